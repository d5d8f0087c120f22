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
//
// Warps g, g+FW, ... land on the same SM sub-partition and run the same specialised
// body, so each sub-partition's instruction stream is one compact loop.  The last warp
// of the CTA is the producer: it issues the bulk copies of a tile and stages the tile's
// harmonics and receiver ids.  The warps of a row group compute the group's A entries of
// the next tile right after finishing the current one.
#pragma once
#include "fast_common.cuh"

namespace e3j {
namespace fast {


// Per A slot: up to two records, A = c0 * y[i2_0] + c1 * y[i2_1].
struct ASlot {
    float c0, c1;
    int i2_0, i2_1;
};

template <class S>
struct FwdSmem {
    static constexpr int T = S::FT, NS = S::FS;
    static constexpr int CH = S::NQ / (32 * S::V);
    static constexpr int NCONS = S::FW * CH;       // consumer warps
    static constexpr int S_EDGE = S::P * S::NQ;    // floats of weights per edge
    static constexpr int X_EDGE = S::DIN * S::NQ;  // floats of one sender row
    static constexpr size_t up(size_t v, size_t a) { return (v + a - 1) / a * a; }
    static constexpr size_t off_bar = 0;                                  // full[NS], empty[NS]
    static constexpr size_t off_pair = off_bar + 16 * NS;                 // pair[FW]: a row group's warps have written their A shares
    static constexpr size_t off_abort = off_pair + 8 * S::FW;
    static constexpr size_t off_stage = up(off_abort + 4, 128);
    static constexpr size_t st_s = 0;
    static constexpr size_t st_x = st_s + 4 * (size_t)T * S_EDGE;
    static constexpr size_t st_A = st_x + 4 * (size_t)T * X_EDGE;         // float A[T][APAD]
    static constexpr size_t st_y = st_A + 4 * (size_t)T * S::F_APAD;
    static constexpr size_t st_r = st_y + 4 * (size_t)T * S::DSH;         // recv[T], change mask
    static constexpr size_t stage_bytes = up(st_r + 4 * (T + 1), 128);
    static constexpr size_t total = off_stage + NS * stage_bytes;
};

// ------------------------------------------------------------------------ consumer
template <class S, int G>
__device__ __forceinline__ void fwd_consumer(const FwdParams& p, unsigned char* smem, const int ch, const int warp,
                                             const int lane, const int64_t e_begin, const int64_t e_end,
                                             const int n_tiles) {
    using Vec = typename VecOf<S::V>::type;
    using L = FwdSmem<S>;
    constexpr int T = L::T, NS = L::NS;
    constexpr int NQV = S::NQ / S::V;
    constexpr int ROW0 = S::f_row0(G), ROW1 = S::f_row0(G + 1);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* empty = full + NS;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    const int cta = blockIdx.x;
    const int vlane = ch * 32 + lane;
    const int64_t row_elems = (int64_t)S::D * S::NQ;
    // identity mode: receiver of edge e is e, so no row ever straddles a CTA boundary
    const int prev_recv = p.identity ? (int)e_begin - 1
                                     : ((e_begin > 0 && e_begin < e_end) ? p.receivers[e_begin - 1] : -1);
    const int next_recv = p.identity ? (int)e_end : ((e_end < p.n_edges) ? p.receivers[e_end] : -2);
    if (!p.identity && warp == 0 && lane == 0) { p.part_recv[2 * cta] = -1; p.part_recv[2 * cta + 1] = -1; }

    // The CH warps of row group G share the group's A entries of a tile: each lane of the
    // CH*32 computes entries idx = pl, pl + CH*32, ... (entry idx -> edge idx / NP, slot idx % NP).
    constexpr int A0 = S::f_a0(G), NP = S::f_a0(G + 1) - A0;
    constexpr int NI = (T * NP + L::CH * 32 - 1) / (L::CH * 32);
    ASlot a_tab[NI];
    int a_dst[NI];
    {
        const int pl = ch * 32 + lane;
#pragma unroll
        for (int i = 0; i < NI; ++i) {
            const int idx = pl + L::CH * 32 * i;
            const bool valid = idx < T * NP;
            const int e_i = valid ? idx / NP : 0, slot = A0 + (valid ? idx % NP : 0);
            const PairRec pr = S::pair_rec(slot);
            ASlot a{0.f, 0.f, 0, 0};
            if (valid && pr.count > 0) { a.c0 = S::rec_val(pr.start); a.i2_0 = e_i * S::DSH + S::rec_i2(pr.start); }
            if (valid && pr.count > 1) { a.c1 = S::rec_val(pr.start + 1); a.i2_1 = e_i * S::DSH + S::rec_i2(pr.start + 1); }
            a_tab[i] = a;
            a_dst[i] = valid ? e_i * S::F_APAD + slot : -1;
        }
    }
    // A[e][slot] = sum over the slot's records of c * y[e][i2] for one landed tile
    // (entries of edges beyond the tile's length are computed from stale data and never read)
    uint64_t* pair = reinterpret_cast<uint64_t*>(smem + L::off_pair) + G;
    int pair_phase = 0;
    auto make_A = [&](unsigned char* st) -> bool {
        const float* y_t = reinterpret_cast<const float*>(st + L::st_y);
        float* A_t = reinterpret_cast<float*>(st + L::st_A);
#pragma unroll
        for (int i = 0; i < NI; ++i)
            if (a_dst[i] >= 0)
                A_t[a_dst[i]] = (fmaf(a_tab[i].c1, y_t[a_tab[i].i2_1], a_tab[i].c0 * y_t[a_tab[i].i2_0]));
        __syncwarp();
        if constexpr (L::CH > 1) {
            // the group's other warps hold the rest of the entries (bounded wait, like every wait here)
            if (lane == 0) mbar_arrive(pair);
            const bool ok = mbar_wait(pair, pair_phase, abort_flag, p.status);
            pair_phase ^= 1;
            return ok;
        }
        return true;
    };

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
    // A finished row goes straight to global memory (its final place, or this CTA's partial-row slot).
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
        S::template fwd_store<G>(acc, reinterpret_cast<Vec*>(base) + (size_t)ROW0 * NQV + vlane, NQV);
    };
    auto new_receiver = [&](const int r) {
        if (cur >= 0) { flush(false); seg_first = false; }
        zero_rows((cur >= 0 ? cur : prev_recv) + 1, r);
        cur = r;
#pragma unroll
        for (int q = 0; q < S::F_RMAX; ++q) vzero(acc[q]);
    };

    int stage = 0, phase = 0;                 // ring slot of tile t and the parity of its use
    int left = (int)(e_end - e_begin);        // edges of this CTA not yet consumed
    bool ok = n_tiles > 0 && mbar_wait(&full[0], 0, abort_flag, p.status);
    if (ok) ok = make_A(smem + L::off_stage);
    for (int t = 0; ok && t < n_tiles; ++t) {
        const unsigned char* st = smem + L::off_stage + stage * (int)L::stage_bytes;
        const int n_e = min(T, left);
        left -= T;
        const int* recv_t = reinterpret_cast<const int*>(st + L::st_r);
        unsigned mask = (unsigned)recv_t[T];  // bit i: edge i starts a new receiver
        const Vec* xs = reinterpret_cast<const Vec*>(st + L::st_x) + vlane;
        const Vec* ss = reinterpret_cast<const Vec*>(st + L::st_s) + vlane;
        const float* As = reinterpret_cast<const float*>(st + L::st_A);
        // one compact body per edge: a longer (unrolled) loop costs more in instruction fetch than it saves
#pragma unroll 1
        for (int e_i = 0; e_i < n_e; ++e_i) {
            if (mask & 1u) new_receiver(recv_t[e_i]);
            mask >>= 1;
            S::template fwd_edge<G>(acc, xs, ss, As);
            xs += L::X_EDGE / S::V; ss += L::S_EDGE / S::V; As += S::F_APAD;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[stage]);
        if (++stage == NS) { stage = 0; phase ^= 1; }
        if (t + 1 < n_tiles) {
            // next tile: wait for its data, then this warp's share of its A entries
            ok = mbar_wait(&full[stage], phase, abort_flag, p.status);
            if (ok) ok = make_A(smem + L::off_stage + stage * (int)L::stage_bytes);
        }
    }
    if (!*abort_flag) {
        if (cur >= 0) {
            flush(true);
            if (e_end == p.n_edges && !p.identity) zero_rows(cur + 1, (int)p.n_nodes);
        }
    }
}

template <class S, int G>
struct FwdDispatch {
    template <class... Args>
    __device__ static __forceinline__ void run(const int g, Args&&... args) {
        if (g == G) fwd_consumer<S, G>(args...);
        else FwdDispatch<S, G + 1>::run(g, args...);
    }
};
template <class S>
struct FwdDispatch<S, S::FW> {
    template <class... Args>
    __device__ static __forceinline__ void run(const int, Args&&...) {}
};

// ------------------------------------------------------------------------ producer
template <class S>
__device__ __forceinline__ void fwd_producer(const FwdParams& p, unsigned char* smem, const int warp, const int lane,
                                             const int64_t e_begin, const int64_t e_end, const int n_tiles) {
    using L = FwdSmem<S>;
    constexpr int T = L::T, NS = L::NS;
    constexpr int YPL = (T * S::DSH + 31) / 32;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* empty = full + NS;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    int snd_a = 0, rcv_a = -1, snd_b = 0, rcv_b = -1;
    float y_a[YPL], y_b[YPL];
    auto load_meta = [&](int t, int& snd, int& rcv, float (&yv)[YPL]) {
        if (t >= n_tiles) return;
        const int64_t e0 = e_begin + (int64_t)t * T;
        const int n_e = (int)min((int64_t)T, e_end - e0);
        if (lane < n_e) {
            if (p.identity) { snd = rcv = (int)(e0 + lane); }
            else { snd = p.senders[e0 + lane]; rcv = p.receivers[e0 + lane]; }
        }
#pragma unroll
        for (int i = 0; i < YPL; ++i) {
            const int idx = i * 32 + lane;
            if (idx < n_e * S::DSH) yv[i] = p.sh[e0 * S::DSH + idx];
        }
    };
    load_meta(0, snd_a, rcv_a, y_a);
    load_meta(1, snd_b, rcv_b, y_b);
    int armed = 0, last_rcv = -1, stage = 0, phase = 0;
    for (int t = 0; t < n_tiles; ++t) {
        // phase of `empty` that ends the previous use of this ring slot
        if (t >= NS && !mbar_wait(&empty[stage], phase ^ 1, abort_flag, p.status)) break;
        unsigned char* st = smem + L::off_stage + stage * (int)L::stage_bytes;
        const int64_t e0 = e_begin + (int64_t)t * T;
        const int n_e = (int)min((int64_t)T, e_end - e0);
        int* recv_t = reinterpret_cast<int*>(st + L::st_r);
        float* y_t = reinterpret_cast<float*>(st + L::st_y);
        // copies first: they are the long pole
        if (lane == 0) {
            mbar_expect_tx(&full[stage], (uint32_t)n_e * (uint32_t)(4 * (L::S_EDGE + L::X_EDGE)));
            bulk_g2s(st + L::st_s, p.w + (size_t)e0 * L::S_EDGE, (uint32_t)n_e * 4u * L::S_EDGE, &full[stage]);
        }
        if (lane < n_e)
            bulk_g2s(st + L::st_x + (size_t)lane * 4 * L::X_EDGE, p.x + (size_t)snd_a * L::X_EDGE, 4u * L::X_EDGE,
                     &full[stage]);
        armed = t + 1;
        int before = __shfl_up_sync(0xffffffffu, rcv_a, 1);
        if (lane == 0) before = last_rcv;
        const unsigned mask = __ballot_sync(0xffffffffu, lane < n_e && rcv_a != before);
        last_rcv = __shfl_sync(0xffffffffu, rcv_a, n_e - 1);
        if (lane < n_e) recv_t[lane] = rcv_a;
        if (lane == 0) recv_t[T] = (int)mask;
#pragma unroll
        for (int i = 0; i < YPL; ++i) {
            const int idx = i * 32 + lane;
            if (idx < n_e * S::DSH) y_t[idx] = y_a[i];
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&full[stage]);  // the staged harmonics / receiver ids are in place
        snd_a = snd_b; rcv_a = rcv_b;
#pragma unroll
        for (int i = 0; i < YPL; ++i) y_a[i] = y_b[i];
        load_meta(t + 2, snd_b, rcv_b, y_b);
        if (++stage == NS) { stage = 0; phase ^= 1; }
    }
    if (*abort_flag) {
        // let copies already in flight land before the CTA's shared memory is released
        for (int t = max(0, armed - NS); t < armed; ++t)
            for (uint32_t it = 0; it < kSpinLimit; ++it)
                if (mbar_try_wait(&full[t % NS], (t / NS) & 1)) break;
    }
}

template <class S>
__global__ void __launch_bounds__((S::FW * (S::NQ / (32 * S::V)) + 1) * 32, S::FC)
fast_fwd_kernel(const FwdParams p) {
    using L = FwdSmem<S>;
    constexpr int T = L::T, NS = L::NS, NCONS = L::NCONS;
    static_assert(T <= 31, "the change mask is one 32-bit word");
    static_assert(S::F_NREC <= 2, "an A slot holds at most two records");

    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* empty = full + NS;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t e_begin = min(p.n_edges, (int64_t)blockIdx.x * p.chunk);
    const int64_t e_end = min(p.n_edges, e_begin + p.chunk);
    const int n_tiles = (int)((e_end - e_begin + T - 1) / T);

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], NCONS); }
        for (int g = 0; g < S::FW; ++g) mbar_init(reinterpret_cast<uint64_t*>(smem + L::off_pair) + g, L::CH);
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    if (warp == NCONS) fwd_producer<S>(p, smem, warp, lane, e_begin, e_end, n_tiles);
    else FwdDispatch<S, 0>::run(warp % S::FW, p, smem, warp / S::FW, warp, lane, e_begin, e_end, n_tiles);
}

}  // namespace fast
}  // namespace e3j
