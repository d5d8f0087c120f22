// Signature-specialised forward convolution kernel (template over a generated struct S).
//
// Work split: the receiver-sorted edge list is cut into one contiguous range per CTA
// (equal edge counts, so every SM streams the same number of bytes).  A CTA walks its
// range in tiles of S::FT edges; warp (g, ch) owns output rows
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
    static constexpr int A_WARP = T * S::F_APAD + 32;  // A floats per channel chunk (+ dummy slots)
    static constexpr size_t up(size_t v, size_t a) { return (v + a - 1) / a * a; }
    static constexpr size_t off_bar = 0;                                  // full[NS], empty[NS]
    static constexpr size_t off_abort = off_bar + 16 * NS;
    static constexpr size_t off_A = up(off_abort + 4, 16);                // float[CH][A_WARP]
    static constexpr size_t off_stage = up(off_A + 4 * CH * A_WARP, 128);
    static constexpr size_t st_s = 0;
    static constexpr size_t st_x = st_s + 4 * (size_t)T * S_EDGE;
    static constexpr size_t st_y = st_x + 4 * (size_t)T * X_EDGE;
    static constexpr size_t st_r = st_y + 4 * (size_t)T * S::DSH;         // recv[T], change mask
    static constexpr size_t stage_bytes = up(st_r + 4 * (T + 1), 128);
    static constexpr size_t total = off_stage + NS * stage_bytes;
};

// One warp: row group G, channel chunk ch.  Warps g, g+FW, ... land on the same SM
// sub-partition and run the same code, which keeps the instruction stream of a
// sub-partition to one specialised body.
//
// There is no dedicated producer warp: the warp whose index equals (tile mod warps)
// refills a stage (after every warp has released it) with the tile NS steps ahead.
template <class S, int G>
__device__ __forceinline__ void fwd_warp(const FwdParams& p, unsigned char* smem, const int ch, const int warp,
                                         const int lane, const int64_t e_begin, const int64_t e_end,
                                         const int n_tiles) {
    using Vec = typename VecOf<S::V>::type;
    using L = FwdSmem<S>;
    constexpr int T = L::T, NS = L::NS, NW = S::FW * L::CH;
    constexpr int NQV = S::NQ / S::V;
    constexpr int A0 = S::f_a0(G), NP = S::f_a0(G + 1) - A0;
    constexpr int ROW0 = S::f_row0(G), ROW1 = S::f_row0(G + 1);
    constexpr int NI = (T * NP + 31) / 32;   // A entries computed per lane and tile
    constexpr int NR = S::F_NREC;            // records per (i0,i1) pair, at most
    constexpr int YPL = (T * S::DSH + 31) / 32;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* empty = full + NS;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    float* A_w = reinterpret_cast<float*>(smem + L::off_A) + (size_t)ch * L::A_WARP;
    const int cta = blockIdx.x;
    const int vlane = ch * 32 + lane;
    const int64_t row_elems = (int64_t)S::D * S::NQ;
    const int prev_recv = (e_begin > 0 && e_begin < e_end) ? p.receivers[e_begin - 1] : -1;
    const int next_recv = (e_end < p.n_edges) ? p.receivers[e_end] : -2;
    if (warp == 0 && lane == 0) { p.part_recv[2 * cta] = -1; p.part_recv[2 * cta + 1] = -1; }

    // ---- refill duty: metadata of the next tile this warp will issue, prefetched in registers
    int duty = warp, m_snd = 0, m_rcv = -1, m_before = -1;
    float m_y[YPL];
    auto load_meta = [&](int u) {
        if (u >= n_tiles) return;
        const int64_t e0 = e_begin + (int64_t)u * T;
        const int n_e = (int)min((int64_t)T, e_end - e0);
        if (lane < n_e) { m_snd = p.senders[e0 + lane]; m_rcv = p.receivers[e0 + lane]; }
        m_before = (u > 0) ? p.receivers[e0 - 1] : -1;
#pragma unroll
        for (int i = 0; i < YPL; ++i) {
            const int idx = i * 32 + lane;
            if (idx < n_e * S::DSH) m_y[i] = p.sh[e0 * S::DSH + idx];
        }
    };
    auto issue = [&](int u) {
        const int stage = u % NS;
        unsigned char* st = smem + L::off_stage + (size_t)stage * L::stage_bytes;
        const int64_t e0 = e_begin + (int64_t)u * T;
        const int n_e = (int)min((int64_t)T, e_end - e0);
        int* recv_t = reinterpret_cast<int*>(st + L::st_r);
        float* y_t = reinterpret_cast<float*>(st + L::st_y);
        int before = __shfl_up_sync(0xffffffffu, m_rcv, 1);
        if (lane == 0) before = m_before;
        const unsigned mask = __ballot_sync(0xffffffffu, lane < n_e && m_rcv != before);
        if (lane < n_e) recv_t[lane] = m_rcv;
        if (lane == 0) recv_t[T] = (int)mask;
#pragma unroll
        for (int i = 0; i < YPL; ++i) {
            const int idx = i * 32 + lane;
            if (idx < n_e * S::DSH) y_t[idx] = m_y[i];
        }
        __syncwarp();
        if (lane == 0) {
            mbar_arrive_expect_tx(&full[stage], (uint32_t)n_e * (uint32_t)(4 * (L::S_EDGE + L::X_EDGE)));
            bulk_g2s(st + L::st_s, p.w + (size_t)e0 * L::S_EDGE, (uint32_t)n_e * 4u * L::S_EDGE, &full[stage]);
        }
        if (lane < n_e)
            bulk_g2s(st + L::st_x + (size_t)lane * 4 * L::X_EDGE, p.x + (size_t)m_snd * L::X_EDGE, 4u * L::X_EDGE,
                     &full[stage]);
    };
    load_meta(duty);
    if (duty < NS && duty < n_tiles) { issue(duty); duty += NW; load_meta(duty); }

    // ---- this lane's share of the tile's A entries: A[dst] = sum_r coef[r] * y_tile[src[r]]
    float a_coef[NI][NR];
    int a_src[NI][NR], a_dst[NI];
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        const int idx = lane + 32 * i;
        const bool valid = idx < T * NP;
        const int e_i = valid ? idx / NP : 0, slot = A0 + (valid ? idx % NP : 0);
        const PairRec pr = S::pair_rec(slot);
        a_dst[i] = valid ? e_i * S::F_APAD + slot : T * S::F_APAD + lane;
#pragma unroll
        for (int r = 0; r < NR; ++r) {
            const bool on = valid && r < pr.count;
            a_coef[i][r] = on ? S::rec_val(pr.start + r) : 0.f;
            a_src[i][r] = on ? e_i * S::DSH + S::rec_i2(pr.start + r) : 0;
        }
    }

    Vec acc[S::F_RMAX];
#pragma unroll
    for (int r = 0; r < S::F_RMAX; ++r) vzero(acc[r]);
    int cur = -1;
    bool seg_first = true;
    Vec zero; vzero(zero);

    auto zero_rows = [&](int lo, int hi) {  // receivers lo..hi-1 have no edges
        for (int b = lo; b < hi; ++b) {
            Vec* dst = reinterpret_cast<Vec*>(p.out + (size_t)b * row_elems) + vlane;
#pragma unroll
            for (int row = ROW0; row < ROW1; ++row) dst[(size_t)row * NQV] = zero;
        }
    };
    auto flush = [&](bool at_end) {
        const bool head = seg_first && cur == prev_recv;
        const bool tail = at_end && cur == next_recv;
        float* base;
        if (head) {
            base = p.partial + (size_t)(2 * cta) * row_elems;
            if (warp == 0 && lane == 0) p.part_recv[2 * cta] = cur;
        } else if (tail) {
            base = p.partial + (size_t)(2 * cta + 1) * row_elems;
            if (warp == 0 && lane == 0) p.part_recv[2 * cta + 1] = cur;
        } else {
            base = p.out + (size_t)cur * row_elems;
        }
        S::template fwd_store<G>(acc, reinterpret_cast<Vec*>(base) + vlane);
    };

    for (int t = 0; t < n_tiles; ++t) {
        const int stage = t % NS, use = t / NS;
        if (!mbar_wait(&full[stage], use & 1, abort_flag, p.status)) break;
        const unsigned char* st = smem + L::off_stage + (size_t)stage * L::stage_bytes;
        const int n_e = (int)min((int64_t)T, e_end - (e_begin + (int64_t)t * T));
        const int* recv_t = reinterpret_cast<const int*>(st + L::st_r);
        const float* y_t = reinterpret_cast<const float*>(st + L::st_y);
        // entries of edges beyond n_e are computed from stale data and never read
#pragma unroll
        for (int i = 0; i < NI; ++i) {
            float a = 0.f;
#pragma unroll
            for (int r = 0; r < NR; ++r) a = fmaf(a_coef[i][r], y_t[a_src[i][r]], a);
            A_w[a_dst[i]] = a;
        }
        const int mask = recv_t[T];  // bit i: edge i starts a new receiver
        __syncwarp();
        const Vec* xs = reinterpret_cast<const Vec*>(st + L::st_x) + vlane;
        const Vec* ss = reinterpret_cast<const Vec*>(st + L::st_s) + vlane;
        const float* As = A_w;
#pragma unroll 1  // the body is long straight-line code; unrolling it overflows the instruction cache
        for (int e_i = 0; e_i < n_e; ++e_i) {
            if ((mask >> e_i) & 1) {
                const int r = recv_t[e_i];
                if (cur >= 0) { flush(false); seg_first = false; }
                zero_rows((cur >= 0 ? cur : prev_recv) + 1, r);
                cur = r;
#pragma unroll
                for (int q = 0; q < S::F_RMAX; ++q) vzero(acc[q]);
            }
            S::template fwd_edge<G>(acc, xs, ss, As);
            xs += L::X_EDGE / S::V; ss += L::S_EDGE / S::V; As += S::F_APAD;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[stage]);
        if (t + NS == duty && duty < n_tiles) {
            // every warp has released this stage once empty's phase `use` completes
            if (!mbar_wait(&empty[stage], use & 1, abort_flag, p.status)) break;
            issue(duty);
            duty += NW;
            load_meta(duty);
        }
    }
    if (!*abort_flag) {
        if (cur >= 0) {
            flush(true);
            if (e_end == p.n_edges) zero_rows(cur + 1, (int)p.n_nodes);
        }
    } else {
        // give copies that are still in flight time to land before shared memory is released
        for (int i = 0; i < 64; ++i) __nanosleep(2000);
    }
}

template <class S, int G>
struct FwdDispatch {
    template <class... Args>
    __device__ static __forceinline__ void run(const int g, Args&&... args) {
        if (g == G) fwd_warp<S, G>(args...);
        else FwdDispatch<S, G + 1>::run(g, args...);
    }
};
template <class S>
struct FwdDispatch<S, S::FW> {
    template <class... Args>
    __device__ static __forceinline__ void run(const int, Args&&...) {}
};

template <class S>
__global__ void __launch_bounds__(S::FW * (S::NQ / (32 * S::V)) * 32, S::FC)
fast_fwd_kernel(const FwdParams p) {
    using L = FwdSmem<S>;
    constexpr int T = L::T, NS = L::NS, NW = S::FW * L::CH;
    static_assert(T <= 31, "the change mask is one 32-bit word");
    static_assert(NS <= NW, "one warp refills one stage at a time");

    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* empty = full + NS;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t e_begin = min(p.n_edges, (int64_t)blockIdx.x * p.chunk);
    const int64_t e_end = min(p.n_edges, e_begin + p.chunk);
    const int n_tiles = (int)((e_end - e_begin + T - 1) / T);

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], NW); }
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    FwdDispatch<S, 0>::run(warp % S::FW, p, smem, warp / S::FW, warp, lane, e_begin, e_end, n_tiles);
}

}  // namespace fast
}  // namespace e3j
