// Forward convolution that forms its edge scalars inside the kernel from the radial network's last layer,
// s[e, k, q] = sum_j h[e, j] W[j, k N_q + q], so that the [E, P, N_q] weight array never exists in memory.
//
// The product needs W next to the tensor cores for every edge, and W (hidden x P N_q floats, twice for the TF32
// split) is larger than one SM's shared memory.  The convolution is independent per channel, so the work is cut
// by CHANNELS: a CTA owns kCS = 16 channels (its 106 KB slice of W stays resident) and one range of the edge
// list; eight CTAs with neighbouring block ids cover the 128 channels of the same range.
//
// Slots.  The edges of every receiver are padded to a multiple of 8 "slots" (slot tables: fast_radial.cu); a
// group of 8 slots x 16 channels is laid out as 128 "virtual channels" (lane l of a consumer warp = slot l % 8,
// channel quad l / 8), which is exactly the shape of one edge x 128 channels of the plain forward kernel: the
// generated per-edge bodies S::fwd_edge<G> run unchanged, only their A pointer differs per lane (A belongs to the
// slot).  When the receiver changes, the 8 slot lanes are added with three shuffle steps (fixed order) and
// the row is stored; rows cut by a range boundary go to the partial-row scratch and fwd_fixup_kernel.
//
// Per tile of 128 slots (16 groups):
//   converter warps   h rows of the tile's edges -> (hi, lo) TF32 -> tensor memory (A operand, lane = slot)
//   MMA warp          D[slot, (k, q)] = h W_slice, three tcgen05.mma passes of hidden / 8 steps each, N = P * 16
//   epilogue warps    D (tensor memory, lane = slot) -> shared-memory stage in the virtual-channel layout
//   producer warp     sender rows (16-channel pieces), A entries from the harmonics, receiver ids -> same stage
//   consumer warps    the convolution body over the stage's groups, one warp per row group
// Stages hold a quarter tile (4 groups); two stages.  Every wait is bounded.
#pragma once
#include "../umma.cuh"
#include "fast_common.cuh"

namespace e3j {
namespace fast {

constexpr int kCS = 16;          // channels per CTA
constexpr int kGroup = 8;        // slots per group (lanes of one channel quad)
constexpr int kTileSlots = 128;  // slots per tensor-core tile
constexpr int kQuarterSlots = 32;
constexpr int kRadialThreads = 14 * 32;
constexpr int kMaxHidden = 64;

struct RadialFwdParams {
    const float* x; const float* sh; const float* h; const float* W;
    const int32_t* senders;
    const int32_t* slotptr; const int32_t* slot_edge; const int32_t* group_recv;
    float* out;
    float* partial; int32_t* part_recv;   // [n_ranges][2][D * NQ], [n_ranges][2]
    int32_t* status;
    int64_t n_nodes;
    int hidden, n_ranges;
};

template <class S>
struct RadialSmem {
    static constexpr int NROW = S::P * kCS;                      // rows of the W slice = N of the product
    static constexpr int ASTR = S::F_APAD + 4;                   // floats between the A entries of two slots
    static_assert(ASTR % 32 == 4 || ASTR % 32 == 12 || ASTR % 32 == 20 || ASTR % 32 == 28,
                  "A rows of the 8 slots of a group must start in different banks");
    static constexpr size_t w_bytes = (size_t)NROW * kMaxHidden * 4;        // one of hi / lo
    static constexpr size_t st_s = 0;                                         // [4][P][128] floats
    static constexpr size_t st_x = st_s + 4 * (size_t)4 * S::P * 128;         // [4][DIN][128]
    static constexpr size_t st_A = st_x + 4 * (size_t)4 * S::DIN * 128;       // [32][ASTR]
    static constexpr size_t st_meta = st_A + 4 * (size_t)kQuarterSlots * ASTR; // recv[4], n_valid
    static constexpr size_t stage_bytes = (st_meta + 32 + 127) / 128 * 128;
    static constexpr size_t off_bar = 0;   // stage_full[2], q_empty[4], h_full[2], h_empty[2], d_full, d_empty, drain
    static constexpr size_t off_tmem = 8 * 13;
    static constexpr size_t off_abort = off_tmem + 4;
    static constexpr size_t off_w = 1024;
    static constexpr size_t off_stage = off_w + 2 * w_bytes;
    static constexpr size_t total = off_stage + 2 * stage_bytes;
    // tensor memory columns
    static constexpr uint32_t col_d = 0, col_h = 256, tmem_cols = 512;   // h buffer b: hi at col_h + 128 b, lo 64 further
};

// Bounded wait that records WHICH wait gave up: the first failure stores `code` (role in the low byte, tile or
// quarter index above it) in the status word.
__device__ __forceinline__ bool rwait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status, int code) {
#pragma unroll 1
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    if (status) atomicCAS(status, 0, code);
    return false;
}

// sum over the 8 slot lanes of a channel quad (lane bits 0..2), same order on every lane
__device__ __forceinline__ float4 sum_slots(float4 v) {
#pragma unroll
    for (int m = 1; m < 8; m <<= 1) {
        v.x += __shfl_xor_sync(0xffffffffu, v.x, m);
        v.y += __shfl_xor_sync(0xffffffffu, v.y, m);
        v.z += __shfl_xor_sync(0xffffffffu, v.z, m);
        v.w += __shfl_xor_sync(0xffffffffu, v.w, m);
    }
    return v;
}

// ------------------------------------------------------------------------ consumer (one warp per row group)
template <class S, int G>
__device__ __forceinline__ void radial_consumer(const RadialFwdParams& p, unsigned char* smem, const int lane,
                                                const int cg, const int range, const int g_begin, const int g_end,
                                                const int n_groups, const int n_quarters) {
    using L = RadialSmem<S>;
    using Vec = float4;
    constexpr int NQV = S::NQ / 4;
    constexpr int ROW0 = S::f_row0(G), ROW1 = S::f_row0(G + 1);
    uint64_t* stage_full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* q_empty = stage_full + 2;   // one per quarter position of a tile
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    const int j = lane & 7, quad = lane >> 3;
    const int64_t row_elems = (int64_t)S::D * S::NQ;
    const int prev_recv = (g_begin > 0 && g_begin < g_end) ? p.group_recv[g_begin - 1] : -1;
    const int next_recv = (g_end < n_groups) ? p.group_recv[g_end] : -2;
    if (G == 0 && cg == 0 && lane == 0) { p.part_recv[2 * range] = -1; p.part_recv[2 * range + 1] = -1; }

    Vec acc[S::F_RMAX];
#pragma unroll
    for (int r = 0; r < S::F_RMAX; ++r) vzero(acc[r]);
    int cur = -1;
    bool seg_first = true;
    const Vec zero = make_float4(0.f, 0.f, 0.f, 0.f);

    auto zero_rows = [&](int lo, int hi) {   // receivers lo..hi-1 have no edges
        if (j != 0) return;
        for (int b = lo; b < hi; ++b) {
            Vec* dst = reinterpret_cast<Vec*>(p.out + (size_t)b * row_elems) + cg * (kCS / 4) + quad;
#pragma unroll
            for (int row = ROW0; row < ROW1; ++row) dst[(size_t)row * NQV] = zero;
        }
    };
    auto flush = [&](bool at_end) {
#pragma unroll
        for (int r = 0; r < ROW1 - ROW0; ++r) acc[r] = sum_slots(acc[r]);
        const bool head = seg_first && cur == prev_recv;
        const bool tail = at_end && cur == next_recv;
        float* base;
        if (head) {
            base = p.partial + (size_t)(2 * range) * row_elems;
            if (G == 0 && cg == 0 && lane == 0) p.part_recv[2 * range] = cur;
        } else if (tail) {
            base = p.partial + (size_t)(2 * range + 1) * row_elems;
            if (G == 0 && cg == 0 && lane == 0) p.part_recv[2 * range + 1] = cur;
        } else {
            base = p.out + (size_t)cur * row_elems;
        }
        if (j == 0)
            S::template fwd_store<G>(acc, reinterpret_cast<Vec*>(base) + (size_t)ROW0 * NQV + cg * (kCS / 4) + quad, NQV);
    };
    auto new_receiver = [&](const int r) {
        if (cur >= 0) { flush(false); seg_first = false; }
        zero_rows((cur >= 0 ? cur : prev_recv) + 1, r);
        cur = r;
#pragma unroll
        for (int q = 0; q < S::F_RMAX; ++q) vzero(acc[q]);
    };

    for (int qi = 0; qi < n_quarters; ++qi) {
        const int stage = qi & 1;
        if (!rwait(&stage_full[stage], (qi >> 1) & 1, abort_flag, p.status, 0x40 + G + (qi << 8))) break;
        const unsigned char* st = smem + L::off_stage + (size_t)stage * L::stage_bytes;
        const int* meta = reinterpret_cast<const int*>(st + L::st_meta);   // recv[4], n_valid, change mask
        const int n_valid = meta[4];
        unsigned mask = (unsigned)meta[5];
        const Vec* xs = reinterpret_cast<const Vec*>(st + L::st_x) + lane;
        const Vec* ss = reinterpret_cast<const Vec*>(st + L::st_s) + lane;
        const float* As = reinterpret_cast<const float*>(st + L::st_A) + j * L::ASTR;
        int gq = 0;
        while (gq < n_valid) {
            if (mask & 1u) new_receiver(meta[gq]);
            mask >>= 1;
            const int run = min(mask ? __ffs((int)mask) : 4, n_valid - gq);
            mask >>= run - 1;
            gq += run;
#pragma unroll 1
            for (int i = 0; i < run; ++i) {
                S::template fwd_edge<G>(acc, xs, ss, As);
                xs += S::DIN * NQV; ss += S::P * NQV; As += kGroup * L::ASTR;
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&q_empty[qi & 3]);
    }
    if (!*abort_flag) {
        if (cur >= 0) {
            flush(true);
            if (g_end == n_groups) zero_rows(cur + 1, (int)p.n_nodes);
        }
        if (n_groups == 0 && range == 0) zero_rows(0, (int)p.n_nodes);
    }
}

template <class S, int G>
struct RadialDispatch {
    template <class... Args>
    __device__ static __forceinline__ void run(const int g, Args&&... args) {
        if (g == G) radial_consumer<S, G>(args...);
        else RadialDispatch<S, G + 1>::run(g, args...);
    }
};
template <class S>
struct RadialDispatch<S, S::FW> {
    template <class... Args>
    __device__ static __forceinline__ void run(const int, Args&&...) {}
};

// ------------------------------------------------------------------------ producer warp (lane = slot of the quarter)
template <class S>
__device__ __forceinline__ void radial_producer(const RadialFwdParams& p, unsigned char* smem, const int lane,
                                                const int cg, const int g_begin, const int g_end, const int n_quarters) {
    using L = RadialSmem<S>;
    uint64_t* stage_full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* q_empty = stage_full + 2;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    const int gq = lane >> 3, j = lane & 7;
    int last_recv = -1;
#pragma unroll 1
    for (int qi = 0; qi < n_quarters; ++qi) {
        const int stage = qi & 1;
        // the stage's previous occupant, quarter qi - 2, must have been consumed
        if (qi >= 2 && !rwait(&q_empty[(qi - 2) & 3], ((qi - 2) >> 2) & 1, abort_flag, p.status, 0x50 + (qi << 8))) break;
        unsigned char* st = smem + L::off_stage + (size_t)stage * L::stage_bytes;
        const int g0 = g_begin + 4 * qi;
        const int n_valid = max(0, min(4, g_end - g0));
        const int edge = (gq < n_valid) ? p.slot_edge[(size_t)g0 * kGroup + lane] : -1;
        // A entries of this lane's slot from its harmonics (zero for a padding slot)
        float y[S::DSH];
#pragma unroll
        for (int i = 0; i < S::DSH; ++i) y[i] = (edge >= 0) ? p.sh[(size_t)edge * S::DSH + i] : 0.f;
        S::a_entries(y, reinterpret_cast<float4*>(st + L::st_A) + (size_t)lane * (L::ASTR / 4));
        // the slot's sender row, this CTA's 16 channels of every input coordinate
        const int snd = (edge >= 0) ? p.senders[edge] : 0;
        const float4* src = reinterpret_cast<const float4*>(p.x + ((size_t)snd * S::DIN) * S::NQ + cg * kCS);
        float4 xv[S::DIN][4];
#pragma unroll
        for (int i1 = 0; i1 < S::DIN; ++i1)
#pragma unroll
            for (int qd = 0; qd < 4; ++qd)
                xv[i1][qd] = (edge >= 0) ? src[i1 * (S::NQ / 4) + qd] : make_float4(0.f, 0.f, 0.f, 0.f);
        float4* xdst = reinterpret_cast<float4*>(st + L::st_x) + (size_t)gq * S::DIN * 32 + j;
#pragma unroll
        for (int i1 = 0; i1 < S::DIN; ++i1)
#pragma unroll
            for (int qd = 0; qd < 4; ++qd) xdst[i1 * 32 + qd * 8] = xv[i1][qd];
        // receiver ids of the quarter's groups and where the receiver changes
        const int r = (lane < n_valid) ? p.group_recv[g0 + lane] : -1;
        int before = __shfl_up_sync(0xffffffffu, r, 1);
        if (lane == 0) before = last_recv;
        const unsigned mask = __ballot_sync(0xffffffffu, lane < n_valid && r != before);
        if (n_valid > 0) last_recv = __shfl_sync(0xffffffffu, r, n_valid - 1);
        int* meta = reinterpret_cast<int*>(st + L::st_meta);
        if (lane < 4) meta[lane] = r;
        if (lane == 0) { meta[4] = n_valid; meta[5] = (int)mask; }
        __syncwarp();
        if (lane == 0) mbar_arrive(&stage_full[stage]);
    }
}

// ------------------------------------------------------------------------ the kernel
template <class S>
__global__ void __launch_bounds__(kRadialThreads, 1) radial_fwd_kernel(const RadialFwdParams p) {
    using L = RadialSmem<S>;
    static_assert(S::V == 4 && S::FW == 4, "the bodies must be the four-channel, four-row-group ones");
    static_assert(L::NROW % 16 == 0 && L::NROW <= 256, "N of the product");
    static_assert(L::total <= 227 * 1024, "shared memory");
    constexpr int NCG = S::NQ / kCS;
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* stage_full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* q_empty = stage_full + 2;
    uint64_t* h_full = q_empty + 4;
    uint64_t* h_empty = h_full + 2;
    uint64_t* d_full = h_empty + 2;
    uint64_t* d_empty = d_full + 1;
    uint64_t* drain = d_empty + 1;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::off_tmem);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cg = blockIdx.x % NCG, range = blockIdx.x / NCG;
    const int H = p.hidden;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) { mbar_init(&stage_full[s], 2); mbar_init(&h_full[s], 4); mbar_init(&h_empty[s], 1); }
        for (int q = 0; q < 4; ++q) mbar_init(&q_empty[q], S::FW);
        mbar_init(d_full, 1); mbar_init(d_empty, 4); mbar_init(drain, 1);
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 13) umma::tmem_alloc(tmem_slot, L::tmem_cols);
    // this CTA's slice of W, split into TF32 pairs, K-major: row r = k * 16 + channel, K = hidden
    {
        unsigned char* w_hi = smem + L::off_w;
        unsigned char* w_lo = w_hi + L::w_bytes;
        const int quads = H / 4;
        for (int idx = threadIdx.x; idx < L::NROW * quads; idx += kRadialThreads) {
            const int r = idx % L::NROW, quad = idx / L::NROW;
            const size_t col = (size_t)(r / kCS) * S::NQ + cg * kCS + r % kCS;
            const size_t ldw = (size_t)S::P * S::NQ;
            const float* src = p.W + (size_t)(4 * quad) * ldw + col;
            const float4 v = make_float4(src[0], src[ldw], src[2 * ldw], src[3 * ldw]);
            float4 hi, lo;
            umma::split_tf32(v, hi, lo);
            const uint32_t off = umma::tile_offset(r, 4 * quad, H);
            *reinterpret_cast<float4*>(w_hi + off) = hi;
            *reinterpret_cast<float4*>(w_lo + off) = lo;
        }
        umma::fence_smem_to_async();
    }
    umma::fence_before_sync();
    __syncthreads();
    umma::fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    // the groups of this CTA: whole tiles of 16 groups, equal tile counts per range
    const int n_groups = p.slotptr[p.n_nodes] / kGroup;
    const int tiles_total = (n_groups + 15) / 16;
    const int tiles_per = (tiles_total + p.n_ranges - 1) / p.n_ranges;
    const int t0 = min(tiles_total, range * tiles_per), t1 = min(tiles_total, t0 + tiles_per);
    const int g_begin = 16 * t0, g_end = min(n_groups, 16 * t1);
    const int n_tiles = t1 - t0, n_quarters = 4 * n_tiles;

    if (warp < 4) {
        // -------------------------------------------- epilogue: quarter `warp` of every tile, lane = slot
        const int gq = lane >> 3, j = lane & 7;
#pragma unroll 1
        for (int t = 0; t < n_tiles; ++t) {
            const int qi = 4 * t + warp, stage = warp & 1;
            if (!rwait(d_full, t & 1, abort_flag, p.status, 0x10 + warp + (t << 8))) break;
            umma::fence_after_sync();
            // The stage's previous occupant, quarter qi - 2, must have been consumed.  There is one `empty` barrier
            // per quarter position of a tile, so that every waiter sees each barrier's phases one after the other
            // (a parity wait is only meaningful within one phase of the barrier's current one).
            if (qi >= 2 && !rwait(&q_empty[(qi - 2) & 3], ((qi - 2) >> 2) & 1, abort_flag, p.status, 0x20 + warp + (t << 8))) break;
            unsigned char* st = smem + L::off_stage + (size_t)stage * L::stage_bytes;
            float* sdst = reinterpret_cast<float*>(st + L::st_s) + (size_t)gq * S::P * 128 + j * 4;
            const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + L::col_d;
#pragma unroll 1
            for (int k = 0; k < S::P; ++k) {
                float v[16];
                umma::tmem_ld16(taddr + k * kCS, v);
                umma::tmem_ld_wait();
#pragma unroll
                for (int qd = 0; qd < 4; ++qd)
                    *reinterpret_cast<float4*>(sdst + k * 128 + qd * 32) = make_float4(v[4 * qd], v[4 * qd + 1], v[4 * qd + 2], v[4 * qd + 3]);
            }
            umma::fence_before_sync();
            __syncwarp();
            if (lane == 0) { mbar_arrive(d_empty); mbar_arrive(&stage_full[stage]); }
        }
    } else if (warp < 8) {
        // -------------------------------------------- converters: h rows -> (hi, lo) -> tensor memory, lane = slot
        const int cw = warp - 4;
#pragma unroll 1
        for (int t = 0; t < n_tiles; ++t) {
            const int hb = t & 1;
            if (t >= 2 && !rwait(&h_empty[hb], ((t >> 1) + 1) & 1, abort_flag, p.status, 0x30 + cw + (t << 8))) break;
            const int64_t slot = (int64_t)(g_begin + 16 * t) * kGroup + cw * 32 + lane;
            const int edge = (slot < (int64_t)g_end * kGroup) ? p.slot_edge[slot] : -1;
            const uint32_t taddr = tmem_base + ((uint32_t)(cw * 32) << 16) + L::col_h + hb * 128;
#pragma unroll 1
            for (int half = 0; half < 2; ++half) {
                if (32 * half >= H) break;
                float hi[32], lo[32];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int k = 32 * half + 4 * i;
                    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (edge >= 0 && k < H) v = *reinterpret_cast<const float4*>(p.h + (size_t)edge * H + k);
                    float4 a, b;
                    umma::split_tf32(v, a, b);
                    hi[4 * i] = a.x; hi[4 * i + 1] = a.y; hi[4 * i + 2] = a.z; hi[4 * i + 3] = a.w;
                    lo[4 * i] = b.x; lo[4 * i + 1] = b.y; lo[4 * i + 2] = b.z; lo[4 * i + 3] = b.w;
                }
                umma::tmem_st32(taddr + 32 * half, hi);
                umma::tmem_st32(taddr + 64 + 32 * half, lo);
            }
            umma::tmem_st_wait();
            umma::fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&h_full[hb]);
        }
    } else if (warp < 12) {
        RadialDispatch<S, 0>::run(warp - 8, p, smem, lane, cg, range, g_begin, g_end, n_groups, n_quarters);
    } else if (warp == 12) {
        radial_producer<S>(p, smem, lane, cg, g_begin, g_end, n_quarters);
    } else {
        // -------------------------------------------- tensor-core issue
        constexpr uint32_t idesc = umma::idesc_tf32(kTileSlots, L::NROW);
        const uint32_t sbo = umma::sbo_bytes(H);
        const int ksteps = H / 8;
        const uint32_t w_hi = umma::smem_addr(smem + L::off_w), w_lo = w_hi + (uint32_t)L::w_bytes;
#pragma unroll 1
        for (int t = 0; t < n_tiles; ++t) {
            const int hb = t & 1;
            if (!rwait(&h_full[hb], (t >> 1) & 1, abort_flag, p.status, 0x60 + (t << 8))) break;
            if (t >= 1 && !rwait(d_empty, (t - 1) & 1, abort_flag, p.status, 0x61 + (t << 8))) break;
            umma::fence_after_sync();
            if (lane == 0) {
                const uint32_t a_hi = tmem_base + L::col_h + hb * 128, a_lo = a_hi + 64;
                const uint32_t d = tmem_base + L::col_d;
                const uint32_t pa[3] = {a_lo, a_hi, a_hi}, pb[3] = {w_hi, w_lo, w_hi};   // small terms first
#pragma unroll
                for (int pass = 0; pass < 3; ++pass)
#pragma unroll 1
                    for (int ks = 0; ks < ksteps; ++ks)
                        umma::mma_tf32_ts(d, pa[pass] + ks * 8, umma::make_desc(pb[pass] + ks * 2 * umma::kLbo, umma::kLbo, sbo),
                                          idesc, (pass > 0 || ks > 0) ? 1u : 0u);
                umma::commit(&h_empty[hb]);
                umma::commit(d_full);
            }
            __syncwarp();
        }
        if (*abort_flag) {   // let products in flight finish before tensor memory is freed
            if (lane == 0) umma::commit(drain);
            __syncwarp();
#pragma unroll 1
            for (uint32_t spin = 0; spin < kSpinLimit; ++spin)
                if (mbar_try_wait(drain, 0)) break;
        }
    }
    umma::fence_before_sync();
    __syncthreads();
    if (warp == 13) umma::tmem_dealloc(tmem_base, L::tmem_cols);
}

// ------------------------------------------------------------------------ host side
// Slot tables of a graph (integer kernels, fast_radial.cu): slotptr [n_nodes + 1], slot_edge [slot capacity],
// group_recv [slot capacity / 8]; slot capacity = radial_slot_capacity(n_nodes, n_edges).
inline int64_t radial_slot_capacity(int64_t n_nodes, int64_t n_edges) {
    return (n_edges + (kGroup - 1) * n_nodes + kGroup - 1) / kGroup * kGroup + kGroup;
}
int build_slot_tables(int64_t n_nodes, int64_t n_edges, const int32_t* rowptr, int32_t* slotptr, int32_t* slot_edge,
                      int32_t* group_recv, cudaStream_t st);

template <class S>
size_t radial_fwd_scratch_need(int n_ranges) {
    return kPartRecvBytes + sizeof(float) * 2 * (size_t)n_ranges * S::D * S::NQ;
}

template <class S>
int launch_radial_fwd(const ConvArgs& a, const RadialArgs& r) {
    using L = RadialSmem<S>;
    constexpr int NCG = S::NQ / kCS;
    if (r.hidden % 8 != 0 || r.hidden > kMaxHidden) return E3J_ERR_UNSUPPORTED;   // the caller materialises instead
    const int n_ranges = std::max(1, sm_count() / NCG);
    if (r.scratch_bytes < radial_fwd_scratch_need<S>(n_ranges)) return E3J_ERR_WORKSPACE;
    static thread_local int attr_dev = -1;
    int dev = 0;
    E3J_CUDA_TRY(cudaGetDevice(&dev));
    if (attr_dev != dev) {
        E3J_CUDA_TRY(cudaFuncSetAttribute(radial_fwd_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::total));
        attr_dev = dev;
    }
    RadialFwdParams p{};
    p.x = a.x; p.sh = a.sh; p.h = r.h; p.W = r.W; p.senders = a.senders;
    p.slotptr = r.slotptr; p.slot_edge = r.slot_edge; p.group_recv = r.group_recv;
    p.out = a.out;
    p.part_recv = reinterpret_cast<int32_t*>(r.scratch);
    p.partial = reinterpret_cast<float*>(reinterpret_cast<char*>(r.scratch) + kPartRecvBytes);
    p.status = a.status;
    p.n_nodes = a.n_nodes; p.hidden = r.hidden; p.n_ranges = n_ranges;
    radial_fwd_kernel<S><<<n_ranges * NCG, kRadialThreads, L::total, a.stream>>>(p);
    if (int s = after_launch()) return s;
    fwd_fixup_kernel<<<n_ranges, 256, 0, a.stream>>>(n_ranges, S::D * S::NQ / 4, reinterpret_cast<const float4*>(p.partial),
                                                    p.part_recv, reinterpret_cast<float4*>(a.out));
    return after_launch();
}

}  // namespace fast
}  // namespace e3j
