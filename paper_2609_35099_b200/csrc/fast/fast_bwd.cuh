// Signature-specialised backward convolution, pass 1 (template over a generated struct S).
//
// One sweep over the receiver-sorted edges computes the three cotangents of the paper's
// message-passing-backward equation in the factored form of its "Backward sweep of one
// edge tile":  with A[i0,i1] = sum_{i2} C y[i2] and k the path (irreducible block) of i0,
//   u[k,i1]     = sum_{i0 in k} A[i0,i1] * dm[b,i0]            (per channel)
//   grad_w[e,k] = sum_{i1} x[a,i1] * u[k,i1]
//   dx_e[i1]    = sum_k s[e,k] * u[k,i1]                       (this edge's share of grad_x[a])
//   grad_sh[e,i2] = sum_q sum_{pairs} C[i0,i1,i2] * (s[e,k] x[a,i1]) * dm[b,i0]
// grad_w and grad_sh are edge-local and final.  dx_e is written to a scratch array
// [E,d,N_q]; pass 2 (bwd_dx_reduce_kernel) adds the rows of every sender in edge order, so no
// floating-point atomics are needed and the result is bit-reproducible.
//
// Work split: equal contiguous edge ranges per CTA; consumer warp (g, ch) owns the paths of
// group g (whole paths, so grad_w[e,k] is complete inside one warp) and channels
// [ch*32*V, (ch+1)*32*V).  The rows of dm that a warp needs stay in registers while the receiver
// does not change.  Per edge the warps exchange their dx_e and grad_sh partial sums through
// shared memory and add them in a fixed order.  The last warp is the producer (the code shared with the
// forward kernel, run by one warp here): a tile's copies, then its receiver ids and A entries.
#pragma once
#include "fast_common.cuh"
#include "fast_producer.cuh"

namespace e3j {
namespace fast {

struct BwdParams {
    const float* x; const float* sh; const float* w;
    const float* vec;                  // (forward only; always null here)
    const int32_t* senders; const int32_t* receivers;
    const float* grad_out;
    float* grad_sh; float* grad_w;     // grad_sh may be null: computed all the same, not stored
    float* dx_edge;                    // scratch [E][d][N_q]
    int64_t n_nodes, n_edges, chunk;   // chunk = edges per CTA
    int32_t* status;
    int identity;                      // 1: every edge is its own sender and receiver; dx_edge is then grad_x itself
    const int32_t* n_real;             // padded call: device word holding the number of real edges (else null)
    // fused double backward only: cotangents of grad_x, grad_sh, grad_w (laid out like x, sh, w)
    const float* ct_x; const float* ct_sh; const float* ct_w;
};

template <class S>
struct BwdSmem {
    static constexpr bool DBL = false;             // (the producer code is shared with the double-backward forward)
    static constexpr int T = S::BT, NS = S::BS;
    static constexpr int CH = S::NQ / (32 * S::BV);
    static constexpr int NCONS = S::BW * CH;
    static constexpr int S_EDGE = S::P * S::NQ;
    static constexpr int X_EDGE = S::DIN * S::NQ;
    static constexpr int DYP = 16;                 // grad_sh partial sums per warp (d' padded)
    static_assert(S::DSH <= DYP, "harmonics beyond l = 3 need a wider reduction");
    static constexpr size_t up(size_t v, size_t a) { return (v + a - 1) / a * a; }
    static constexpr size_t off_bar = 0;
    static constexpr size_t off_xch = off_bar + 16 * NS;                               // exchange barrier
    static constexpr size_t off_abort = off_xch + 8;
    static constexpr size_t off_dxs = up(off_abort + 4, 128);                        // float[2][BW][DIN][NQ]
    static constexpr size_t off_dyp = off_dxs + 4 * 2 * (size_t)S::BW * X_EDGE;      // float[2][NCONS][DYP]
    static constexpr size_t off_stage = up(off_dyp + 4 * 2 * (size_t)NCONS * DYP, 128);
    static constexpr size_t st_s = 0;
    static constexpr size_t st_x = st_s + 4 * (size_t)T * S_EDGE;
    static constexpr size_t st_A = st_x + 4 * (size_t)T * X_EDGE;
    static constexpr size_t st_y = st_A + 4 * (size_t)T * S::B_APAD;
    static constexpr size_t st_r = st_y + 4 * (size_t)T * S::DSH;                    // recv[T], change mask
    static constexpr size_t stage_bytes = up(st_r + 4 * (T + 1), 128);
    static constexpr size_t total = off_stage + NS * stage_bytes;
};

// Sum of v[0..15] over the 32 lanes.  On return lane L holds (in the return value) the total
// of entry ((L >> 1) & 15) with bit order (b4 b3 b2 b1) -> entry index b4*8 + b3*4 + b2*2 + b1.
__device__ __forceinline__ float reduce16_over_lanes(float (&v)[16], const int lane) {
    const bool b4 = lane & 16, b3 = lane & 8, b2 = lane & 4, b1 = lane & 2;
    float w8[8], w4[4], w2[2];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float send = b4 ? v[j] : v[j + 8], keep = b4 ? v[j + 8] : v[j];
        w8[j] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float send = b3 ? w8[j] : w8[j + 4], keep = b3 ? w8[j + 4] : w8[j];
        w4[j] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const float send = b2 ? w4[j] : w4[j + 2], keep = b2 ? w4[j + 2] : w4[j];
        w2[j] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    }
    const float send = b1 ? w2[0] : w2[1], keep = b1 ? w2[1] : w2[0];
    float r = keep + __shfl_xor_sync(0xffffffffu, send, 2);
    r += __shfl_xor_sync(0xffffffffu, r, 1);
    return r;
}

// The loop, the exchange and the reductions below are the same instructions for every path group; only
// S::bwd_edge's body differs (chosen by a switch on g), which keeps the kernel's hot code small enough
// for the SM's instruction cache.
template <class S>
__device__ __forceinline__ void bwd_consumer(const BwdParams& p, unsigned char* smem, const int G, const int ch,
                                             const int warp, const int lane, const int64_t e_begin,
                                             const int64_t e_end, const int n_tiles) {
    using Vec = typename S::BVec;
    using L = BwdSmem<S>;
    constexpr int T = L::T, NS = L::NS, NCONS = L::NCONS;
    constexpr int NQV = S::NQ / S::BV;
    const int NROW = S::b_nrow(G);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* empty = full + NS;
    uint64_t* xch = reinterpret_cast<uint64_t*>(smem + L::off_xch);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    float* dxs = reinterpret_cast<float*>(smem + L::off_dxs);
    float* dyp = reinterpret_cast<float*>(smem + L::off_dyp);
    const int vlane = ch * 32 + lane;
    const int64_t row_elems = (int64_t)S::D * S::NQ;

    Vec dm[S::B_RMAX];   // this warp's rows of grad_out[receiver]
#pragma unroll
    for (int r = 0; r < S::B_RMAX; ++r) vzero(dm[r]);

    int stage = 0, phase = 0, buf = 0, xphase = 0;
    bool alive = true;
    int left = (int)(e_end - e_begin);
    int64_t e = e_begin;
    for (int t = 0; alive && t < n_tiles; ++t) {
        if (!mbar_wait(&full[stage], phase, abort_flag, p.status)) break;
        const unsigned char* st = smem + L::off_stage + stage * (int)L::stage_bytes;
        const int n_e = min(T, left);
        left -= T;
        const int* recv_t = reinterpret_cast<const int*>(st + L::st_r);
        unsigned mask = (unsigned)recv_t[T];
        const Vec* xs = reinterpret_cast<const Vec*>(st + L::st_x) + vlane;
        const Vec* ss = reinterpret_cast<const Vec*>(st + L::st_s) + vlane;
        const float* As = reinterpret_cast<const float*>(st + L::st_A);
#pragma unroll 1
        for (int e_i = 0; alive && e_i < n_e; ++e_i, ++e) {
            if (mask & 1u) {
                const Vec* g = reinterpret_cast<const Vec*>(p.grad_out + (size_t)recv_t[e_i] * row_elems) + vlane;
#pragma unroll
                for (int r = 0; r < S::B_RMAX; ++r)
                    if (r < NROW) dm[r] = g[(size_t)S::b_row(G, r) * NQV];  // rows of this warp's path group
            }
            mask >>= 1;
            Vec dxp[S::DIN];   // both are assigned (not accumulated into) by bwd_edge
            float dyl[16];
            Vec* gw = p.grad_w ? reinterpret_cast<Vec*>(p.grad_w + (size_t)e * L::S_EDGE) + vlane : nullptr;   // null: not wanted
            S::bwd_edge(G, dm, xs, ss, As, dxp, dyl, gw);
            xs += L::X_EDGE / S::BV; ss += L::S_EDGE / S::BV; As += S::B_APAD;

            // this warp's partial sums -> shared memory
            const float dy_tot = reduce16_over_lanes(dyl, lane);
            if ((lane & 1) == 0) {
                const int idx = ((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1);
                dyp[(buf * NCONS + warp) * L::DYP + idx] = dy_tot;
            }
            Vec* my = reinterpret_cast<Vec*>(dxs + (size_t)(buf * S::BW + G) * L::X_EDGE) + vlane;
#pragma unroll
            for (int i = 0; i < S::DIN; ++i) my[i * NQV] = dxp[i];
            // every consumer warp has deposited its partial sums (bounded wait, like every other wait here)
            __syncwarp();
            if (lane == 0) mbar_arrive(xch);
            alive = mbar_wait(xch, xphase, abort_flag, p.status);
            xphase ^= 1;
            if (!alive) break;
            // fixed-order sums over the path groups / warps; rows and entries are dealt out to the warps
            for (int i1 = G; i1 < S::DIN; i1 += S::BW) {
                Vec sum; vzero(sum);
#pragma unroll
                for (int g2 = 0; g2 < S::BW; ++g2)
                    sum = vadd(sum, reinterpret_cast<const Vec*>(dxs + (size_t)(buf * S::BW + g2) * L::X_EDGE)[i1 * NQV + vlane]);
                reinterpret_cast<Vec*>(p.dx_edge + (size_t)e * L::X_EDGE)[i1 * NQV + vlane] = sum;
            }
            if (warp == 0 && lane < S::DSH) {
                float sum = 0.f;
#pragma unroll
                for (int w2 = 0; w2 < NCONS; ++w2) sum += dyp[(buf * NCONS + w2) * L::DYP + lane];
                if (p.grad_sh) p.grad_sh[(size_t)e * S::DSH + lane] = sum;
            }
            buf ^= 1;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[stage]);
        if (++stage == NS) { stage = 0; phase ^= 1; }
    }
}

template <class S>
struct BwdTab {
    static constexpr int APAD = S::B_APAD, DSH = S::DSH;
    __device__ static __forceinline__ PairRec pair_rec(int i) { return S::b_pair_rec(i); }
    __device__ static __forceinline__ float rec_val(int i) { return S::b_rec_val(i); }
    __device__ static __forceinline__ unsigned char rec_i2(int i) { return S::b_rec_i2(i); }
};

template <class S>
__global__ void __launch_bounds__((S::BW * (S::NQ / (32 * S::BV)) + 1) * 32, S::BC)
fast_bwd_kernel(const BwdParams p) {
    using L = BwdSmem<S>;
    constexpr int T = L::T, NS = L::NS, NCONS = L::NCONS;
    static_assert(T <= 31, "the change mask is one 32-bit word");
    static_assert(S::B_NREC <= 2, "an A slot holds at most two records");

    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* empty = full + NS;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int64_t n_edges, chunk, e_begin, e_end;   // n_edges: the real edges (a padded call learns their number here)
    cta_edge_range(p.n_edges, p.chunk, p.n_real, n_edges, chunk, e_begin, e_end);
    const int n_tiles = (int)((e_end - e_begin + T - 1) / T);

    if (threadIdx.x == 0) {
        // full: the producer's arrival with the copies' byte count and its arrival after the tables
        for (int s = 0; s < NS; ++s) { mbar_init(&full[s], 2); mbar_init(&empty[s], NCONS); }
        mbar_init(reinterpret_cast<uint64_t*>(smem + L::off_xch), NCONS);
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    if (warp == NCONS) producer_loop<L, BwdTab<S>, 2>(p, smem, lane, e_begin, e_end, n_tiles);
    else bwd_consumer<S>(p, smem, warp % S::BW, warp / S::BW, warp, lane, e_begin, e_end, n_tiles);
}

}  // namespace fast
}  // namespace e3j
