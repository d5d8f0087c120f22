// Signature-specialised forward convolution kernel (template over a generated struct S).
//
// Work split: the receiver-sorted edge list is cut into one contiguous range per CTA
// (equal edge counts, so every SM streams the same number of bytes).  A CTA walks its
// range in tiles of S::FT edges; consumer warp (g, ch) owns output rows
// [S::f_row0(g), S::f_row0(g+1)) and channels [ch*32*V, (ch+1)*32*V) and keeps their
// running sum for the current receiver in registers.  When the receiver changes the
// sum is stored (paper, forward algorithm: accumulate over the receiver's edges, store
// once).  A receiver whose edges straddle a CTA boundary is stored as partial sums
// that fwd_fixup_kernel adds in CTA order, so the result does not depend on timing.
//
// Per edge, the coupling coefficients are contracted with the harmonics once, into
// A[i0,i1] = sum_{i2} C[i0,i1,i2] y[i2] (warp-uniform, kept in shared memory); the
// per-channel work is then acc[i0] += A[i0,i1] * (s[k] * x[i1]) with s factored out of
// the path sum (paper, "Factoring out the edge scalar").
#pragma once
#include "fast_common.cuh"

namespace e3j {
namespace fast {

template <class S>
struct FwdSmem {
    static constexpr int T = S::FT, NS = S::FS;
    static constexpr int CH = S::NQ / (32 * S::V);
    static constexpr int S_EDGE = S::P * S::NQ;    // floats of weights per edge
    static constexpr int X_EDGE = S::DIN * S::NQ;  // floats of one sender row
    static constexpr size_t up(size_t v, size_t a) { return (v + a - 1) / a * a; }
    static constexpr size_t off_bar = 0;                                  // full[NS], empty[NS]
    static constexpr size_t off_abort = off_bar + 16 * NS;
    static constexpr size_t off_pair = up(off_abort + 4, 16);             // PairRec[APAD]
    static constexpr size_t off_val = up(off_pair + 4 * S::F_APAD, 16);   // float[NNZ]
    static constexpr size_t off_i2 = off_val + 4 * S::NNZ;                // uint8[NNZ]
    static constexpr size_t off_A = up(off_i2 + S::NNZ, 16);              // float[CH][T][APAD]
    static constexpr size_t off_stage = up(off_A + 4 * CH * T * S::F_APAD, 128);
    static constexpr size_t st_s = 0;
    static constexpr size_t st_x = st_s + 4 * (size_t)T * S_EDGE;
    static constexpr size_t st_y = st_x + 4 * (size_t)T * X_EDGE;
    static constexpr size_t st_r = st_y + 4 * (size_t)T * S::DSH;
    static constexpr size_t stage_bytes = up(st_r + 4 * T, 128);
    static constexpr size_t total = off_stage + NS * stage_bytes;
};

template <class S>
__global__ void __launch_bounds__((S::FW * (S::NQ / (32 * S::V)) + 1) * 32, S::FC)
fast_fwd_kernel(const FwdParams p) {
    using Vec = typename VecOf<S::V>::type;
    using L = FwdSmem<S>;
    constexpr int T = L::T, NS = L::NS, CH = L::CH;
    constexpr int NQV = S::NQ / S::V;
    constexpr int NCONS = S::FW * CH;
    constexpr int YPL = (T * S::DSH + 31) / 32;

    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* empty = full + NS;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    PairRec* pair_rec = reinterpret_cast<PairRec*>(smem + L::off_pair);
    float* rec_val = reinterpret_cast<float*>(smem + L::off_val);
    uint8_t* rec_i2 = smem + L::off_i2;
    float* A_s = reinterpret_cast<float*>(smem + L::off_A);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = blockIdx.x;
    const int64_t e_begin = min(p.n_edges, (int64_t)cta * p.chunk);
    const int64_t e_end = min(p.n_edges, e_begin + p.chunk);
    const int n_tiles = (int)((e_end - e_begin + T - 1) / T);

    for (int i = threadIdx.x; i < S::F_APAD; i += blockDim.x) pair_rec[i] = S::pair_rec(i);
    for (int i = threadIdx.x; i < S::NNZ; i += blockDim.x) { rec_val[i] = S::rec_val(i); rec_i2[i] = S::rec_i2(i); }
    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], NCONS); }
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        int snd_a = 0, rcv_a = 0, snd_b = 0, rcv_b = 0;
        float y_a[YPL], y_b[YPL];
        auto load_meta = [&](int t, int& snd, int& rcv, float (&yv)[YPL]) {
            if (t >= n_tiles) return;
            const int64_t e0 = e_begin + (int64_t)t * T;
            const int n_e = (int)min((int64_t)T, e_end - e0);
            if (lane < n_e) { snd = p.senders[e0 + lane]; rcv = p.receivers[e0 + lane]; }
#pragma unroll
            for (int i = 0; i < YPL; ++i) {
                const int idx = i * 32 + lane;
                if (idx < n_e * S::DSH) yv[i] = p.sh[e0 * S::DSH + idx];
            }
        };
        load_meta(0, snd_a, rcv_a, y_a);
        load_meta(1, snd_b, rcv_b, y_b);
        int armed = 0;
        for (int t = 0; t < n_tiles; ++t) {
            const int stage = t % NS, use = t / NS;
            if (use > 0 && !mbar_wait(&empty[stage], (use - 1) & 1, abort_flag, p.status)) break;
            unsigned char* st = smem + L::off_stage + (size_t)stage * L::stage_bytes;
            const int64_t e0 = e_begin + (int64_t)t * T;
            const int n_e = (int)min((int64_t)T, e_end - e0);
            int* recv_t = reinterpret_cast<int*>(st + L::st_r);
            float* y_t = reinterpret_cast<float*>(st + L::st_y);
            if (lane < n_e) recv_t[lane] = rcv_a;
#pragma unroll
            for (int i = 0; i < YPL; ++i) {
                const int idx = i * 32 + lane;
                if (idx < n_e * S::DSH) y_t[idx] = y_a[i];
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive_expect_tx(&full[stage], (uint32_t)n_e * (uint32_t)(4 * (L::S_EDGE + L::X_EDGE)));
                bulk_g2s(st + L::st_s, p.w + (size_t)e0 * L::S_EDGE, (uint32_t)n_e * 4u * L::S_EDGE, &full[stage]);
            }
            if (lane < n_e)
                bulk_g2s(st + L::st_x + (size_t)lane * 4 * L::X_EDGE, p.x + (size_t)snd_a * L::X_EDGE,
                         4u * L::X_EDGE, &full[stage]);
            armed = t + 1;
            snd_a = snd_b; rcv_a = rcv_b;
#pragma unroll
            for (int i = 0; i < YPL; ++i) y_a[i] = y_b[i];
            load_meta(t + 2, snd_b, rcv_b, y_b);
        }
        if (*abort_flag) {
            // let copies already in flight land before the CTA's shared memory is released
            for (int t = max(0, armed - NS); t < armed; ++t) {
                for (uint32_t it = 0; it < kSpinLimit; ++it)
                    if (mbar_try_wait(&full[t % NS], (t / NS) & 1)) break;
            }
        }
    } else {
        // ------------------------------------------------------------ consumers
        const int cw = warp - 1, g = cw % S::FW, ch = cw / S::FW;
        const int vlane = ch * 32 + lane;
        const int a0 = S::f_a0(g), np = S::f_a0(g + 1) - a0;
        const int row0 = S::f_row0(g), row1 = S::f_row0(g + 1);
        const int64_t row_elems = (int64_t)S::D * S::NQ;
        const int prev_recv = (e_begin > 0 && e_begin < e_end) ? p.receivers[e_begin - 1] : -1;
        const int next_recv = (e_end < p.n_edges) ? p.receivers[e_end] : -2;
        if (cw == 0 && lane == 0) { p.part_recv[2 * cta] = -1; p.part_recv[2 * cta + 1] = -1; }

        Vec acc[S::F_RMAX];
#pragma unroll
        for (int r = 0; r < S::F_RMAX; ++r) vzero(acc[r]);
        int cur = -1;
        bool seg_first = true;
        Vec zero; vzero(zero);

        auto zero_rows = [&](int lo, int hi) {  // receivers lo..hi-1 have no edges
            for (int b = lo; b < hi; ++b) {
                Vec* dst = reinterpret_cast<Vec*>(p.out + (size_t)b * row_elems) + vlane;
                for (int row = row0; row < row1; ++row) dst[(size_t)row * NQV] = zero;
            }
        };
        auto flush = [&](bool at_end) {
            const bool head = seg_first && cur == prev_recv;
            const bool tail = at_end && cur == next_recv;
            float* base;
            if (head) {
                base = p.partial + (size_t)(2 * cta) * row_elems;
                if (cw == 0 && lane == 0) p.part_recv[2 * cta] = cur;
            } else if (tail) {
                base = p.partial + (size_t)(2 * cta + 1) * row_elems;
                if (cw == 0 && lane == 0) p.part_recv[2 * cta + 1] = cur;
            } else {
                base = p.out + (size_t)cur * row_elems;
            }
            S::fwd_store(g, acc, reinterpret_cast<Vec*>(base) + vlane);
        };

        for (int t = 0; t < n_tiles; ++t) {
            const int stage = t % NS, use = t / NS;
            if (!mbar_wait(&full[stage], use & 1, abort_flag, p.status)) break;
            const unsigned char* st = smem + L::off_stage + (size_t)stage * L::stage_bytes;
            const int64_t e0 = e_begin + (int64_t)t * T;
            const int n_e = (int)min((int64_t)T, e_end - e0);
            const int* recv_t = reinterpret_cast<const int*>(st + L::st_r);
            const float* y_t = reinterpret_cast<const float*>(st + L::st_y);
            float* A_w = A_s + (size_t)ch * T * S::F_APAD;
            // A[pair] = sum_{records of the pair} c * y[i2], for this warp's pairs
            for (int idx = lane; idx < n_e * np; idx += 32) {
                const int e_i = idx / np, j = a0 + (idx - e_i * np);
                const PairRec pr = pair_rec[j];
                float a = 0.f;
                for (int r = pr.start; r < pr.start + pr.count; ++r)
                    a = fmaf(rec_val[r], y_t[e_i * S::DSH + rec_i2[r]], a);
                A_w[e_i * S::F_APAD + j] = a;
            }
            __syncwarp();
#pragma unroll 1
            for (int e_i = 0; e_i < n_e; ++e_i) {
                const int r = recv_t[e_i];
                if (r != cur) {
                    if (cur >= 0) { flush(false); seg_first = false; }
                    zero_rows((cur >= 0 ? cur : prev_recv) + 1, r);
                    cur = r;
#pragma unroll
                    for (int q = 0; q < S::F_RMAX; ++q) vzero(acc[q]);
                }
                const Vec* xs = reinterpret_cast<const Vec*>(st + L::st_x + (size_t)e_i * 4 * L::X_EDGE) + vlane;
                const Vec* ss = reinterpret_cast<const Vec*>(st + L::st_s + (size_t)e_i * 4 * L::S_EDGE) + vlane;
                S::fwd_edge(g, acc, xs, ss, A_w + e_i * S::F_APAD);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[stage]);
        }
        if (!*abort_flag && cur >= 0) {
            flush(true);
            if (e_end == p.n_edges) zero_rows(cur + 1, (int)p.n_nodes);
        }
    }
}

}  // namespace fast
}  // namespace e3j
