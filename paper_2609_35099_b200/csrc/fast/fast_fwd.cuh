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
// body, so each sub-partition's instruction stream is one compact loop.  The last two
// warps of the CTA are producers: one issues the copies of a tile, the other stages the
// tile's receiver ids and computes its A entries, so the consumers' instruction stream
// is the per-edge body and nothing else.
#pragma once
#include "fast_common.cuh"
#include "fast_producer.cuh"

namespace e3j {
namespace fast {


// DBL: the cotangent of grad_out in the double backward, a forward-shaped sum with two terms per coefficient
// pair (S::fwd2_edge); the ring then holds the cotangents (ux, uy -> B, us) beside (x, y -> A, s).
template <class S, bool DBL_ = false>
struct FwdSmem {
    static constexpr bool DBL = DBL_;
    static constexpr int NIN = DBL ? 2 : 1;
    static constexpr int T = DBL ? S::DFT : S::FT, NS = DBL ? S::DFS : S::FS;
    static constexpr int VW = DBL ? S::DFV : S::V;   // channels per lane
    static constexpr int CH = S::NQ / (32 * VW);
    static constexpr int NCONS = S::FW * CH;       // consumer warps
    static constexpr int S_EDGE = S::P * S::NQ;    // floats of weights per edge
    static constexpr int X_EDGE = S::DIN * S::NQ;  // floats of one sender row
    static constexpr size_t up(size_t v, size_t a) { return (v + a - 1) / a * a; }
    static constexpr size_t off_bar = 0;                                  // full[NS], empty[NS]
    static constexpr size_t off_abort = off_bar + 16 * NS;
    static constexpr size_t off_stage = up(off_abort + 4, 128);
    static constexpr size_t st_s = 0;
    static constexpr size_t st_us = st_s + 4 * (size_t)T * S_EDGE;        // (DBL)
    static constexpr size_t st_x = st_s + 4 * (size_t)NIN * T * S_EDGE;
    static constexpr size_t st_ux = st_x + 4 * (size_t)T * X_EDGE;        // (DBL)
    static constexpr size_t st_A = st_x + 4 * (size_t)NIN * T * X_EDGE;   // float A[T][APAD]
    static constexpr size_t st_B = st_A + 4 * (size_t)T * S::F_APAD;      // (DBL)
    static constexpr size_t st_y = st_A + 4 * (size_t)NIN * T * S::F_APAD;
    static constexpr size_t st_uy = st_y + 4 * (size_t)T * S::DSH;        // (DBL)
    static constexpr size_t st_r = st_y + 4 * (size_t)NIN * T * S::DSH;   // recv[T], change mask
    static constexpr size_t stage_bytes = up(st_r + 4 * (T + 1), 128);
    static constexpr size_t total = off_stage + NS * stage_bytes;
};

// ------------------------------------------------------------------------ consumer
template <class S, int G, bool DBL>
__device__ __forceinline__ void fwd_consumer(const FwdParams& p, unsigned char* smem, const int ch, const int warp,
                                             const int lane, const int64_t e_begin, const int64_t e_end,
                                             const int n_tiles, const int64_t n_edges) {
    using L = FwdSmem<S, DBL>;
    using Vec = typename VecOf<L::VW>::type;
    constexpr int T = L::T, NS = L::NS;
    constexpr int NQV = S::NQ / L::VW;
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
    const int next_recv = p.identity ? (int)e_end : ((e_end < n_edges) ? p.receivers[e_end] : -2);
    if (!p.identity && warp == 0 && lane == 0) { p.part_recv[2 * cta] = -1; p.part_recv[2 * cta + 1] = -1; }

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
    for (int t = 0; ok && t < n_tiles; ++t) {
        const unsigned char* st = smem + L::off_stage + stage * (int)L::stage_bytes;
        const int n_e = min(T, left);
        left -= T;
        const int* recv_t = reinterpret_cast<const int*>(st + L::st_r);
        unsigned mask = (unsigned)recv_t[T];  // bit i: edge i starts a new receiver
        const Vec* xs = reinterpret_cast<const Vec*>(st + L::st_x) + vlane;
        const Vec* ss = reinterpret_cast<const Vec*>(st + L::st_s) + vlane;
        const float* As = reinterpret_cast<const float*>(st + L::st_A);
        const Vec* uxs = reinterpret_cast<const Vec*>(st + L::st_ux) + vlane;   // (DBL)
        const Vec* uss = reinterpret_cast<const Vec*>(st + L::st_us) + vlane;
        const float* Bs = reinterpret_cast<const float*>(st + L::st_B);
        // Runs of edges with the same receiver: the inner loop is the bare per-edge body with no receiver
        // test in it (with the test inside, the same body ran 40 % slower), and it is not unrolled (a longer
        // loop costs more in instruction fetch than it saves).
        int e_i = 0;
        while (e_i < n_e) {
            if (mask & 1u) new_receiver(recv_t[e_i]);
            mask >>= 1;                                        // bit 0 now belongs to edge e_i + 1
            const int run = min(mask ? __ffs((int)mask) : T, n_e - e_i);
            mask >>= run - 1;
            e_i += run;
#pragma unroll 1
            for (int j = 0; j < run; ++j) {
                if constexpr (DBL) {
                    S::template fwd2_edge<G>(acc, xs, uxs, ss, uss, As, Bs);
                    uxs += L::X_EDGE / L::VW; uss += L::S_EDGE / L::VW; Bs += S::F_APAD;
                } else {
                    S::template fwd_edge<G>(acc, xs, ss, As);
                }
                xs += L::X_EDGE / L::VW; ss += L::S_EDGE / L::VW; As += S::F_APAD;
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[stage]);
        if (++stage == NS) { stage = 0; phase ^= 1; }
        if (t + 1 < n_tiles) ok = mbar_wait(&full[stage], phase, abort_flag, p.status);
    }
    if (!*abort_flag) {
        if (cur >= 0) {
            flush(true);
            if (e_end == n_edges && !p.identity) zero_rows(cur + 1, (int)p.n_nodes);
        }
        // a padded call without a single real edge: nobody saw a receiver, the first CTA writes the zero rows
        if (n_edges == 0 && cta == 0 && !p.identity) zero_rows(0, (int)p.n_nodes);
    }
}

template <class S, int G, bool DBL>
struct FwdDispatch {
    template <class... Args>
    __device__ static __forceinline__ void run(const int g, Args&&... args) {
        if (g == G) fwd_consumer<S, G, DBL>(args...);
        else FwdDispatch<S, G + 1, DBL>::run(g, args...);
    }
};
template <class S, bool DBL>
struct FwdDispatch<S, S::FW, DBL> {
    template <class... Args>
    __device__ static __forceinline__ void run(const int, Args&&...) {}
};

template <class S>
struct FwdTab {
    static constexpr int APAD = S::F_APAD, DSH = S::DSH;
    __device__ static __forceinline__ PairRec pair_rec(int i) { return S::pair_rec(i); }
    __device__ static __forceinline__ float rec_val(int i) { return S::rec_val(i); }
    __device__ static __forceinline__ unsigned char rec_i2(int i) { return S::rec_i2(i); }
};

template <class S, bool DBL = false>
__global__ void __launch_bounds__((FwdSmem<S, DBL>::NCONS + 2) * 32, DBL ? S::DFC : S::FC)
fast_fwd_kernel(const FwdParams p) {
    using L = FwdSmem<S, DBL>;
    constexpr int T = L::T, NS = L::NS, NCONS = L::NCONS;
    static_assert(T <= 31, "the change mask is one 32-bit word");
    static_assert(S::F_NREC <= 2, "an A slot holds at most two records");

    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* empty = full + NS;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int64_t n_edges, chunk, e_begin, e_end;   // n_edges: the real edges (a padded call learns their number here)
    cta_edge_range(p.n_edges, p.chunk, p.n_real, n_edges, chunk, e_begin, e_end);
    const int n_tiles = (int)((e_end - e_begin + T - 1) / T);

    if (threadIdx.x == 0) {
        // full: the copy warp's arrival (with the byte count) and the table warp's arrival
        for (int s = 0; s < NS; ++s) { mbar_init(&full[s], 2); mbar_init(&empty[s], NCONS); }
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    if (warp == NCONS) producer_loop<L, FwdTab<S>, 0>(p, smem, lane, e_begin, e_end, n_tiles);
    else if (warp == NCONS + 1) producer_loop<L, FwdTab<S>, 1>(p, smem, lane, e_begin, e_end, n_tiles);
    else FwdDispatch<S, 0, DBL>::run(warp % S::FW, p, smem, warp / S::FW, warp, lane, e_begin, e_end, n_tiles, n_edges);
}

}  // namespace fast
}  // namespace e3j
