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
// generated per-edge bodies have the same form, only their A pointer differs per lane (A belongs to the slot).
// When the receiver changes, the 8 slot lanes are added with three shuffle steps (fixed order) and the row is
// stored; rows cut by a range boundary go to the partial-row scratch and fwd_fixup_kernel.
//
// Per tile of 128 slots (16 groups):
//   tile warps (4)    in:  h rows of the tile's edges -> (hi, lo) TF32 -> tensor memory (A operand, lane = slot)
//                     out: D (tensor memory, lane = slot) -> shared-memory stage in the virtual-channel layout
//   MMA warp          D[slot, (k, q)] = h W_slice, three tcgen05.mma passes of hidden / 8 steps each, N = P * 16
//   table warp        A entries from the harmonics, receiver ids -> stage
//   row warp          sender rows (16-channel pieces) -> stage
//   consumer warps    the convolution body over the stage's groups: 4 row groups x 2 warps.  The two warps of a
//                     row group sit on the same SM sub-partition, run the same code (one instruction stream per
//                     sub-partition: with different streams the bodies starve on instruction fetch) and take
//                     alternate groups; at a receiver change the second hands its sums to the first through
//                     shared memory.
// Stages hold a quarter tile (4 groups); two stages.  Registers are moved from the helper warps to the
// consumers (setmaxnreg).  Every wait is bounded.
#pragma once
#include "harmonics.cuh"
#include "../umma.cuh"
#include "fast_common.cuh"

namespace e3j {
namespace fast {

constexpr int kCS = 16;          // channels per CTA
constexpr int kGroup = 8;        // slots per group (lanes of one channel quad)
constexpr int kTileSlots = 128;  // slots per tensor-core tile
constexpr int kQuarterSlots = 32;
constexpr int kMaxHidden = 64;
// warps: 0-3 tile warps, 4-11 consumers (row group (w - 4) % 4, half (w - 4) / 4), 12 tables, 13 tensor-core
// issue, 14 sender rows, 15 idle.  Registers per thread after the prologue: helpers 80 / 96, consumers 168.
constexpr int kRadialThreads = 16 * 32;
constexpr int kRegsTile = 80, kRegsCons = 168, kRegsAux = 96;
static_assert(4 * 32 * (kRegsTile + 2 * kRegsCons + kRegsAux) <= 65536, "register file");

struct RadialFwdParams {
    const float* x; const float* sh; const float* h; const float* W;
    const float* vec;   // edge vectors [E][3]: the table warp forms the harmonics itself (then sh is unused)
    const int32_t* senders;
    const int32_t* slotptr; const int32_t* slot_edge; const int32_t* group_recv;
    float* out;
    float* partial; int32_t* part_recv;   // [n_ranges][2][D * NQ], [n_ranges][2]
    int32_t* status;
    int64_t n_nodes;
    int hidden, n_ranges;
#ifdef E3J_RADIAL_PROF
    unsigned long long* prof;   // 32 counters (cycles per role of CTA 8), zeroed by the caller
#endif
};

template <class S>
struct RadialSmem {
    static_assert(S::R_FW == 4, "one row group per SM sub-partition");
    static constexpr int NROW = S::P * kCS;                      // rows of the W slice = N of the product
    // floats between the A entries of two slots: the rows of the 8 slots of a group must start in different
    // 16-byte bank groups, i.e. the stride is an odd multiple of 4 floats
    static constexpr int astr(int n) { return (n % 8 == 4) ? n : astr(n + 4); }
    static constexpr int ASTR = astr(S::R_APAD);
    static_assert(S::R_APAD % 4 == 0 && ASTR % 8 == 4, "A row stride");
    static constexpr size_t w_bytes = (size_t)NROW * kMaxHidden * 4;        // one of hi / lo
    static constexpr size_t st_s = 0;                                         // [4][P][128] floats
    static constexpr size_t st_x = st_s + 4 * (size_t)4 * S::P * 128;         // [4][DIN][128]
    static constexpr size_t st_A = st_x + 4 * (size_t)4 * S::DIN * 128;       // [32][ASTR]
    static constexpr size_t st_meta = st_A + 4 * (size_t)kQuarterSlots * ASTR; // recv[4], n_valid, change mask
    static constexpr size_t stage_bytes = (st_meta + 32 + 127) / 128 * 128;
    // barriers: stage_full[2], q_empty[4], h_full[2], h_empty[2], d_full, d_empty, drain, xchg[4]
    static constexpr size_t off_bar = 0;
    static constexpr size_t off_tmem = 8 * 17;
    static constexpr size_t off_abort = off_tmem + 4;
    static constexpr size_t off_xchg = 256;   // [4 row groups][2 buffers][16 rows][4 quads] float4
    static constexpr size_t xchg_bytes = (size_t)4 * 2 * 16 * 4 * 16;
    static constexpr size_t off_w = (off_xchg + xchg_bytes + 1023) / 1024 * 1024;
    static constexpr size_t off_stage = off_w + 2 * w_bytes;
    static constexpr size_t total = off_stage + 2 * stage_bytes;
    // tensor memory columns
    static constexpr uint32_t col_d = 0, col_h = 256, tmem_cols = 512;   // h buffer b: hi at col_h + 128 b, lo 64 further
};

// Bounded wait that records WHICH wait gave up: the first failure stores `code` (role in the low byte, tile or
// quarter index above it) in the status word.  Consumers (codes 0x4x) poll back to back; the other roles wait
// for microseconds and sleep between polls.
__device__ __forceinline__ bool rwait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status, int code) {
    const bool relaxed = (code & 0xf0) != 0x40;
#pragma unroll 1
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (relaxed) __nanosleep(64);
        if ((it & 15u) == 15u && *abort_flag) return false;
    }
    *abort_flag = 1;
    if (status) atomicCAS(status, 0, code);
    return false;
}

#ifdef E3J_RADIAL_PROF
#define RPROF_T0 const long long rp_t0 = clock64()
#define RPROF_ADD(slot) do { if (blockIdx.x == 8 && (threadIdx.x & 31) == 0) atomicAdd(&p.prof[slot], (unsigned long long)(clock64() - rp_t0)); } while (0)
#else
#define RPROF_T0
#define RPROF_ADD(slot)
#endif

template <int N> __device__ __forceinline__ void regs_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void regs_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

// ------------------------------------------------------------------------ consumers
// Row group G, warp `half` of its two warps: the groups with (group index & 1) == half.  Both warps see every
// receiver change; there the second warp's sums go through shared memory to the first, which stores the row.
template <class S, int G>
struct RadialBody {   // the generated body of row group g, chosen at run time (warp-uniform)
    __device__ static __forceinline__ void run(const int g, float4 (&acc)[S::R_RMAX], const float4* xs, const float4* ss,
                                               const float* As) {
        if (g == G) S::template rfwd_edge<G>(acc, xs, ss, As);
        else RadialBody<S, G + 1>::run(g, acc, xs, ss, As);
    }
};
template <class S>
struct RadialBody<S, S::R_FW> {
    __device__ static __forceinline__ void run(const int, float4 (&)[S::R_RMAX], const float4*, const float4*, const float*) {}
};

// One function for all row groups: only the per-group bodies differ (RadialBody), everything around them -- the
// loop, the slot reduction, the hand-over between the two warps, the stores -- exists once in the kernel text.
// With one copy per row group the kernel's hot code outgrew the instruction caches and every warp of the SM
// starved on instruction fetch.
template <class S>
__device__ __forceinline__ void radial_consumer(const RadialFwdParams& p, unsigned char* smem, const int lane,
                                                const int G, const int half, const int cg, const int range,
                                                const int g_begin, const int g_end, const int n_groups,
                                                const int n_quarters) {
    using L = RadialSmem<S>;
    using Vec = float4;
    constexpr int NQV = S::NQ / 4;
    const int ROW0 = S::r_row0(G), ROW1 = S::r_row0(G + 1), NR = ROW1 - ROW0;
    static_assert(S::R_RMAX <= 16, "the slot reduction covers 16 rows");
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* stage_full = bars;
    uint64_t* q_empty = bars + 2;   // one per quarter position of a tile
    uint64_t* xbar = bars + 13 + G;
    Vec* xchg = reinterpret_cast<Vec*>(smem + L::off_xchg) + (size_t)G * 2 * 16 * 4;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    const int j = lane & 7, quad = lane >> 3;
    const int64_t row_elems = (int64_t)S::D * S::NQ;
    const int prev_recv = (g_begin > 0 && g_begin < g_end) ? p.group_recv[g_begin - 1] : -1;
    const int next_recv = (g_end < n_groups) ? p.group_recv[g_end] : -2;
    const bool scribe = (G == 0 && cg == 0 && half == 0 && lane == 0);   // writes the boundary receiver ids
    if (scribe) { p.part_recv[2 * range] = -1; p.part_recv[2 * range + 1] = -1; }

    Vec acc[S::R_RMAX];
#pragma unroll
    for (int r = 0; r < S::R_RMAX; ++r) vzero(acc[r]);
    int cur = -1, n_flush = 0;
    bool seg_first = true, ok = true;
    const Vec zero = make_float4(0.f, 0.f, 0.f, 0.f);

    auto zero_rows = [&](int lo, int hi) {   // receivers lo..hi-1 have no edges
        if (j != 0 || half != 0) return;
        for (int b = lo; b < hi; ++b) {
            Vec* dst = reinterpret_cast<Vec*>(p.out + (size_t)b * row_elems) + cg * (kCS / 4) + quad;
            for (int row = ROW0; row < ROW1; ++row) dst[(size_t)row * NQV] = zero;
        }
    };
    auto shfl4 = [](const Vec v, const int m) {
        return make_float4(__shfl_xor_sync(0xffffffffu, v.x, m), __shfl_xor_sync(0xffffffffu, v.y, m),
                           __shfl_xor_sync(0xffffffffu, v.z, m), __shfl_xor_sync(0xffffffffu, v.w, m));
    };
    auto pick = [](const bool c, const Vec a, const Vec b) { return c ? a : b; };
    auto flush = [&](bool at_end) {
        // Sum over the 8 slot lanes of a channel quad (lane bits 0..2) as a reduce-scatter: every step halves the
        // rows a lane carries and exchanges the other half with its partner, so 14 rows cross lanes instead of
        // 3 x NR; afterwards slot lane (b2 b1 b0) holds the complete sums of rows 8 b2 + 4 b1 + 2 b0 + {0, 1}.
        // The order of the additions is fixed by the lane numbers.
        // (rows at and beyond NR are never touched by the body and stay zero)
        const bool b2 = j & 4, b1 = j & 2, b0 = j & 1;
        Vec k8[8], k4[4], k2[2];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const Vec lo = (i < S::R_RMAX) ? acc[i < S::R_RMAX ? i : 0] : zero;
            const Vec hi = (i + 8 < S::R_RMAX) ? acc[i + 8 < S::R_RMAX ? i + 8 : 0] : zero;
            k8[i] = vadd(pick(b2, hi, lo), shfl4(pick(b2, lo, hi), 4));
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) k4[i] = vadd(pick(b1, k8[i + 4], k8[i]), shfl4(pick(b1, k8[i], k8[i + 4]), 2));
#pragma unroll
        for (int i = 0; i < 2; ++i) k2[i] = vadd(pick(b0, k4[i + 2], k4[i]), shfl4(pick(b0, k4[i], k4[i + 2]), 1));
        const int row = (j & 4) * 2 + (j & 2) * 2 + (j & 1) * 2;   // first of this lane's two rows
        // the second warp's sums: two buffers in turn, so that one barrier per flush orders writes and reads
        Vec* buf = xchg + (size_t)(n_flush & 1) * 16 * 4 + row * 4 + quad;
        if (half == 1) { buf[0] = k2[0]; buf[4] = k2[1]; }
        __syncwarp();
        if (lane == 0) mbar_arrive(xbar);
        ok = rwait(xbar, n_flush & 1, abort_flag, p.status, 0x48 + G + (n_flush << 8));
        ++n_flush;
        const bool head = seg_first && cur == prev_recv;
        const bool tail = at_end && cur == next_recv;
        float* base;
        if (head) {
            base = p.partial + (size_t)(2 * range) * row_elems;
            if (scribe) p.part_recv[2 * range] = cur;
        } else if (tail) {
            base = p.partial + (size_t)(2 * range + 1) * row_elems;
            if (scribe) p.part_recv[2 * range + 1] = cur;
        } else {
            base = p.out + (size_t)cur * row_elems;
        }
        if (ok && half == 0) {   // first warp + second warp, then the row's 16 bytes of this channel quad
            Vec* dst = reinterpret_cast<Vec*>(base) + (size_t)(ROW0 + row) * NQV + cg * (kCS / 4) + quad;
            if (row < NR) dst[0] = vadd(k2[0], buf[0]);
            if (row + 1 < NR) dst[NQV] = vadd(k2[1], buf[4]);
        }
    };
    // One instance of this code per row group: the end of the CTA's range is handled as one more receiver change
    // (at_end), and the loops around it are not unrolled -- the flush is long, and copies of it pushed the kernel
    // text beyond what the instruction caches hold (the bodies then starved on instruction fetch).
    auto new_receiver = [&](const int r, const bool at_end) {
        const bool had = cur >= 0;
        if (had) { flush(at_end); seg_first = false; }
        if (!at_end || had) zero_rows((had ? cur : prev_recv) + 1, r);
        cur = r;
#pragma unroll
        for (int q = 0; q < S::R_RMAX; ++q) vzero(acc[q]);
    };

#pragma unroll 1
    for (int qi = 0; ok && qi <= n_quarters; ++qi) {
        const bool last = qi == n_quarters;   // sentinel: flush the last receiver, zero the rows after it
        const int stage = qi & 1;
        RPROF_T0;
        if (!last && !rwait(&stage_full[stage], (qi >> 1) & 1, abort_flag, p.status, 0x40 + G + (qi << 8))) break;
        if (G == 0 && half == 0) RPROF_ADD(8);
        const unsigned char* st = smem + L::off_stage + (size_t)stage * L::stage_bytes;
        const int* meta = reinterpret_cast<const int*>(st + L::st_meta);   // recv[4], n_valid, change mask
        const int n_valid = last ? 1 : meta[4];
        unsigned mask = last ? 1u : (unsigned)meta[5];
        const Vec* xs0 = reinterpret_cast<const Vec*>(st + L::st_x) + lane;
        const Vec* ss0 = reinterpret_cast<const Vec*>(st + L::st_s) + lane;
        const float* As0 = reinterpret_cast<const float*>(st + L::st_A) + j * L::ASTR;
        int gq = 0;
#pragma unroll 1
        while (gq < n_valid) {
            if (mask & 1u) new_receiver(last ? ((g_end == n_groups) ? (int)p.n_nodes : 0) : meta[gq], last);
            mask >>= 1;
            const int run = min(mask ? __ffs((int)mask) : 4, n_valid - gq);
            mask >>= run - 1;
            const int first = gq + ((gq ^ half) & 1);   // this warp's groups of the run
            gq += run;
            const Vec* xs = xs0 + first * (S::DIN * NQV);
            const Vec* ss = ss0 + first * (S::P * NQV);
            const float* As = As0 + first * (kGroup * L::ASTR);
#pragma unroll 1
            for (int g2 = first; g2 < (last ? 0 : gq); g2 += 2) {
                RadialBody<S, 0>::run(G, acc, xs, ss, As);
                xs += 2 * S::DIN * NQV; ss += 2 * S::P * NQV; As += 2 * kGroup * L::ASTR;
            }
        }
        __syncwarp();
        if (!last && lane == 0) mbar_arrive(&q_empty[qi & 3]);
    }
}

// ------------------------------------------------------------------------ stage producers (lane = slot of the quarter)
// Software pipelines: the loads of quarter qi + 1 are issued right after the stores of quarter qi, the slot's
// edge id two quarters ahead (the row warp: three) and its sender id one further back, so that no global-memory
// latency sits between a freed stage and its refill and no load waits on another inside the loop.
template <class S>
struct RadialRange {
    int g_begin, g_end, n_quarters;
    __device__ __forceinline__ int valid_groups(int qi) const { return max(0, min(4, g_end - (g_begin + 4 * qi))); }
    __device__ __forceinline__ int edge_of(const RadialFwdParams& p, int qi, int lane) const {
        return (qi < n_quarters && (lane >> 3) < valid_groups(qi)) ? p.slot_edge[(size_t)(g_begin + 4 * qi) * kGroup + lane] : -1;
    }
};

// A entries from the harmonics, receiver ids and the "receiver changes here" mask
template <class S>
__device__ __forceinline__ void radial_table_warp(const RadialFwdParams& p, unsigned char* smem, const int lane,
                                                  const RadialRange<S> rg) {
    using L = RadialSmem<S>;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* stage_full = bars;
    uint64_t* q_empty = bars + 2;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    float y[S::DSH];
    int recv = -1;
    auto load_data = [&](int qi, int edge) {
        if (p.vec) {
            if (edge >= 0) {
                float ux, uy, uz, inv_r;
                unit_vector(p.vec[(size_t)edge * 3], p.vec[(size_t)edge * 3 + 1], p.vec[(size_t)edge * 3 + 2], ux, uy, uz, inv_r);
                harmonics<S::DSH>(ux, uy, uz, y);
            } else {
#pragma unroll
                for (int i = 0; i < S::DSH; ++i) y[i] = 0.f;
            }
        } else {
#pragma unroll
            for (int i = 0; i < S::DSH; ++i) y[i] = (edge >= 0) ? p.sh[(size_t)edge * S::DSH + i] : 0.f;
        }
        recv = (qi < rg.n_quarters && lane < rg.valid_groups(qi)) ? p.group_recv[rg.g_begin + 4 * qi + lane] : -1;
    };
    load_data(0, rg.edge_of(p, 0, lane));
    int edge1 = rg.edge_of(p, 1, lane);
    int last_recv = -1;
#pragma unroll 1
    for (int qi = 0; qi < rg.n_quarters; ++qi) {
        const int stage = qi & 1;
        RPROF_T0;
        // the stage's previous occupant, quarter qi - 2, must have been consumed
        if (qi >= 2 && !rwait(&q_empty[(qi - 2) & 3], ((qi - 2) >> 2) & 1, abort_flag, p.status, 0x50 + (qi << 8))) break;
        RPROF_ADD(4);
        unsigned char* st = smem + L::off_stage + (size_t)stage * L::stage_bytes;
        const int n_valid = rg.valid_groups(qi);
        S::a_entries(y, reinterpret_cast<float4*>(st + L::st_A) + (size_t)lane * (L::ASTR / 4));   // zero for padding slots
        const int r = recv;
        int before = __shfl_up_sync(0xffffffffu, r, 1);
        if (lane == 0) before = last_recv;
        const unsigned mask = __ballot_sync(0xffffffffu, lane < n_valid && r != before);
        if (n_valid > 0) last_recv = __shfl_sync(0xffffffffu, r, n_valid - 1);
        int* meta = reinterpret_cast<int*>(st + L::st_meta);
        if (lane < 4) meta[lane] = r;
        if (lane == 0) { meta[4] = n_valid; meta[5] = (int)mask; }
        __syncwarp();
        if (lane == 0) mbar_arrive(&stage_full[stage]);
        RPROF_ADD(5);
        load_data(qi + 1, edge1);
        edge1 = rg.edge_of(p, qi + 2, lane);
    }
}

// the slot's sender row: this CTA's 16 channels of every input coordinate
template <class S>
__device__ __forceinline__ void radial_row_warp(const RadialFwdParams& p, unsigned char* smem, const int lane,
                                                const int cg, const RadialRange<S> rg) {
    using L = RadialSmem<S>;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* stage_full = bars;
    uint64_t* q_empty = bars + 2;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    const int gq = lane >> 3, j = lane & 7;
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
    float4 xv[S::DIN][4];
    auto load_rows = [&](int edge, int snd) {
        const float4* src = reinterpret_cast<const float4*>(p.x + ((size_t)snd * S::DIN) * S::NQ + cg * kCS);
#pragma unroll
        for (int i1 = 0; i1 < S::DIN; ++i1)
#pragma unroll
            for (int qd = 0; qd < 4; ++qd) xv[i1][qd] = (edge >= 0) ? src[i1 * (S::NQ / 4) + qd] : zero4;
    };
    auto sender_of = [&](int edge) { return edge >= 0 ? p.senders[edge] : 0; };
    int edge1 = rg.edge_of(p, 0, lane), snd1 = sender_of(edge1);
    load_rows(edge1, snd1);
    edge1 = rg.edge_of(p, 1, lane); snd1 = sender_of(edge1);
    int edge2 = rg.edge_of(p, 2, lane);
#pragma unroll 1
    for (int qi = 0; qi < rg.n_quarters; ++qi) {
        const int stage = qi & 1;
        RPROF_T0;
        if (qi >= 2 && !rwait(&q_empty[(qi - 2) & 3], ((qi - 2) >> 2) & 1, abort_flag, p.status, 0x70 + (qi << 8))) break;
        RPROF_ADD(6);
        unsigned char* st = smem + L::off_stage + (size_t)stage * L::stage_bytes;
        float4* xdst = reinterpret_cast<float4*>(st + L::st_x) + (size_t)gq * S::DIN * 32 + j;
#pragma unroll
        for (int i1 = 0; i1 < S::DIN; ++i1)
#pragma unroll
            for (int qd = 0; qd < 4; ++qd) xdst[i1 * 32 + qd * 8] = xv[i1][qd];
        __syncwarp();
        if (lane == 0) mbar_arrive(&stage_full[stage]);
        RPROF_ADD(7);
        load_rows(edge1, snd1);
        edge1 = edge2; snd1 = sender_of(edge1);
        edge2 = rg.edge_of(p, qi + 3, lane);
    }
}

// ------------------------------------------------------------------------ the kernel
template <class S>
__global__ void __launch_bounds__(kRadialThreads, 1) radial_fwd_kernel(const RadialFwdParams p) {
    using L = RadialSmem<S>;
    static_assert(S::V == 4, "the bodies must be the four-channel ones");
    static_assert(L::NROW % 16 == 0 && L::NROW <= 256, "N of the product");
    static_assert(L::total <= 227 * 1024, "shared memory");
    constexpr int NCG = S::NQ / kCS;
    constexpr int kTableWarp = 12, kMmaWarp = 13, kRowWarp = 14;
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* stage_full = bars;
    uint64_t* q_empty = bars + 2;
    uint64_t* h_full = bars + 6;
    uint64_t* h_empty = bars + 8;
    uint64_t* d_full = bars + 10;
    uint64_t* d_empty = bars + 11;
    uint64_t* drain = bars + 12;
    uint64_t* xbar = bars + 13;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::off_tmem);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    RPROF_T0;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cg = blockIdx.x % NCG, range = blockIdx.x / NCG;
    const int H = p.hidden;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) { mbar_init(&stage_full[s], 3); mbar_init(&h_full[s], 4); mbar_init(&h_empty[s], 1); }
        for (int q = 0; q < 4; ++q) { mbar_init(&q_empty[q], 8); mbar_init(&xbar[q], 2); }
        mbar_init(d_full, 1); mbar_init(d_empty, 4); mbar_init(drain, 1);
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == kMmaWarp) umma::tmem_alloc(tmem_slot, L::tmem_cols);
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
    const RadialRange<S> rg{g_begin, g_end, n_quarters};

    if (warp < 4) {
        // -------------------------------------------- tile warps: quarter `warp` of every tile, lane = slot.
        // In: the slot's row of h, split into TF32 pairs, to tensor memory (A operand of the product), two tiles
        // ahead.  Out: the slot's row of the product from tensor memory to the stage ring.
        regs_dec<kRegsTile>();
        const int gq = lane >> 3, j = lane & 7;
        auto convert = [&](int t) -> bool {
            RPROF_T0;
            const int hb = t & 1;
            if (t >= 2 && !rwait(&h_empty[hb], ((t >> 1) + 1) & 1, abort_flag, p.status, 0x30 + warp + (t << 8))) return false;
            const int64_t slot = (int64_t)(g_begin + 16 * t) * kGroup + warp * 32 + lane;
            const int edge = (slot < (int64_t)g_end * kGroup) ? p.slot_edge[slot] : -1;
            const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + L::col_h + hb * 128;
#pragma unroll 1
            for (int k0 = 0; k0 < H; k0 += 16) {   // 16 columns at a time: the warp has few registers
                float4 v[4];
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    v[i] = (edge >= 0 && k0 + 4 * i < H) ? *reinterpret_cast<const float4*>(p.h + (size_t)edge * H + k0 + 4 * i)
                                                         : make_float4(0.f, 0.f, 0.f, 0.f);
                float hi[16], lo[16];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float4 a, b;
                    umma::split_tf32(v[i], a, b);
                    hi[4 * i] = a.x; hi[4 * i + 1] = a.y; hi[4 * i + 2] = a.z; hi[4 * i + 3] = a.w;
                    lo[4 * i] = b.x; lo[4 * i + 1] = b.y; lo[4 * i + 2] = b.z; lo[4 * i + 3] = b.w;
                }
                umma::tmem_st16(taddr + k0, hi);
                umma::tmem_st16(taddr + 64 + k0, lo);
            }
            umma::tmem_st_wait();
            umma::fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&h_full[hb]);
            if (warp == 0) RPROF_ADD(0);   // convert incl. its wait
            return true;
        };
        // h runs two tiles ahead of the product: step t of the loop moves tile t out and tile t + 2 in
#pragma unroll 1
        for (int t = -2; t < n_tiles; ++t) {
            if (t < 0) {
                if (t + 2 < n_tiles && !convert(t + 2)) break;
                continue;
            }
            const int qi = 4 * t + warp, stage = warp & 1;
            RPROF_T0;
            if (!rwait(d_full, t & 1, abort_flag, p.status, 0x10 + warp + (t << 8))) break;
            umma::fence_after_sync();
            // The stage's previous occupant, quarter qi - 2, must have been consumed.  There is one `empty` barrier
            // per quarter position of a tile, so that every waiter sees each barrier's phases one after the other
            // (a parity wait is only meaningful within one phase of the barrier's current one).
            if (qi >= 2 && !rwait(&q_empty[(qi - 2) & 3], ((qi - 2) >> 2) & 1, abort_flag, p.status, 0x20 + warp + (t << 8))) break;
            if (warp == 0) RPROF_ADD(1);   // waits of the epilogue
            unsigned char* st = smem + L::off_stage + (size_t)stage * L::stage_bytes;
            float* sdst = reinterpret_cast<float*>(st + L::st_s) + (size_t)gq * S::P * 128 + j * 4;
            const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + L::col_d;
#pragma unroll 1
            for (int k = 0; k + 1 < S::P; k += 2) {   // two paths (32 columns) per tensor-memory load
                float v[32];
                umma::tmem_ld32(taddr + k * kCS, v);
                umma::tmem_ld_wait();
#pragma unroll
                for (int kk = 0; kk < 2; ++kk)
#pragma unroll
                    for (int qd = 0; qd < 4; ++qd)
                        *reinterpret_cast<float4*>(sdst + (k + kk) * 128 + qd * 32) =
                            make_float4(v[16 * kk + 4 * qd], v[16 * kk + 4 * qd + 1], v[16 * kk + 4 * qd + 2], v[16 * kk + 4 * qd + 3]);
            }
            if (S::P % 2) {
                constexpr int k = S::P - 1;
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
            if (warp == 0) RPROF_ADD(2);   // epilogue waits + copy
            if (t + 2 < n_tiles && !convert(t + 2)) break;
        }
    } else if (warp < 12) {
        regs_inc<kRegsCons>();
        radial_consumer<S>(p, smem, lane, (warp - 4) & 3, (warp - 4) >> 2, cg, range, g_begin, g_end, n_groups, n_quarters);
    } else {
        regs_dec<kRegsAux>();
        if (warp == kTableWarp) {
            radial_table_warp<S>(p, smem, lane, rg);
        } else if (warp == kRowWarp) {
            radial_row_warp<S>(p, smem, lane, cg, rg);
        } else if (warp == kMmaWarp) {
            // ---------------------------------------- tensor-core issue
            constexpr uint32_t idesc = umma::idesc_tf32(kTileSlots, L::NROW);
            const uint32_t sbo = umma::sbo_bytes(H);
            const int ksteps = H / 8;
            const uint32_t w_hi = umma::smem_addr(smem + L::off_w), w_lo = w_hi + (uint32_t)L::w_bytes;
#pragma unroll 1
            for (int t = 0; t < n_tiles; ++t) {
                const int hb = t & 1;
                RPROF_T0;
                if (!rwait(&h_full[hb], (t >> 1) & 1, abort_flag, p.status, 0x60 + (t << 8))) break;
                RPROF_ADD(10);
                if (t >= 1 && !rwait(d_empty, (t - 1) & 1, abort_flag, p.status, 0x61 + (t << 8))) break;
                RPROF_ADD(11);
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
    }
    umma::fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0) RPROF_ADD(31);
    if (warp == kMmaWarp) umma::tmem_dealloc(tmem_base, L::tmem_cols);
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
    p.x = a.x; p.sh = a.sh; p.vec = a.vec; p.h = r.h; p.W = r.W; p.senders = a.senders;
    p.slotptr = r.slotptr; p.slot_edge = r.slot_edge; p.group_recv = r.group_recv;
    p.out = a.out;
    p.part_recv = reinterpret_cast<int32_t*>(r.scratch);
    p.partial = reinterpret_cast<float*>(reinterpret_cast<char*>(r.scratch) + kPartRecvBytes);
    p.status = a.status;
    p.n_nodes = a.n_nodes; p.hidden = r.hidden; p.n_ranges = n_ranges;
#ifdef E3J_RADIAL_PROF
    p.prof = reinterpret_cast<unsigned long long*>(reinterpret_cast<char*>(r.scratch) + r.scratch_bytes - 65536);
#endif
    radial_fwd_kernel<S><<<n_ranges * NCG, kRadialThreads, L::total, a.stream>>>(p);
    if (int s = after_launch()) return s;
    return launch_dependent(fwd_fixup_kernel, dim3(n_ranges), dim3(256), 0, a.stream, n_ranges, S::D * S::NQ / 4, reinterpret_cast<const float4*>(p.partial),
                                                    p.part_recv, reinterpret_cast<float4*>(a.out));
}

}  // namespace fast
}  // namespace e3j
