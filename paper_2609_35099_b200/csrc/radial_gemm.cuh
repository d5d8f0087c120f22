// Dense products around the radial network's last layer, on the fifth-generation tensor cores (sm_100a).
//
// One kernel template computes C[m, n] = sum_k A[m, k] * B[n, k] for float32 operands with the three-term TF32
// split of umma.cuh.  Output tiles are 128 (m) x N (n = 64 or 128) and live in tensor memory while the K loop
// runs; operands pass through a ring of shared-memory stages of 32 k each, written by converter warps that read
// float32 from global memory, split every value into its (hi, lo) TF32 pair and store both in the K-major
// core-matrix layout that the tensor cores read.  Roles: warps 0-3 read finished tiles out of tensor memory
// and store them, eight warps convert, the last warp issues the tcgen05.mma instructions (one lane).
//
// Where the A operand does not depend on the tile (Prob::A_RESIDENT: the weights product, whose CTA keeps one block
// of W^T for all of its edge tiles) it is converted once into a resident region of shared memory and the stage
// ring carries the B operand alone, with more chunks of loads in flight per converter thread (Prob::PREFETCH).
//
// The two gradient products (Prob::TMA) are built differently, because they read 1 GB each and little else:
//   * One more warp brings the operands in as raw float32 boxes with tiled bulk copies (cp.async.bulk.tensor
//     through a tensor map; rows past the end of a matrix arrive as zeros), a ring of kRawStages boxes deep.  The
//     converter warps read the boxes from shared memory: the loads in flight no longer depend on the converters'
//     registers, and they stay off the load/store pipe.  Boxes whose rows are 128 bytes use the 128-byte
//     swizzle, so that the eight rows a converter quarter-warp reads lie in different banks.
//   * The A operand goes to tensor memory (tcgen05.st, lane = row of the tile) instead of a shared-memory stage:
//     the tensor cores read it without touching shared memory.  The converters are two groups of four warps (one
//     per quarter of the lanes) that take alternate chunks.
//   * A tcgen05.mma of N = 64 is over before its issuing thread has the next one out, so the thread, not the
//     tensor cores, bounds the product.  The three passes are therefore folded into two instructions per k-step:
//     B_hi and B_lo lie behind each other in the stage and serve as one operand of 2 N rows, so that
//     a_hi [b_hi | b_lo] is one instruction, a_lo b_hi the other; two warps issue one of them each, into
//     accumulators of their own (the order of the floating-point sums does not depend on which warp is ahead),
//     and the epilogue adds the three accumulators of a tile, small terms first.
//
// A Problem type describes one product: which output tiles a CTA owns, how many K chunks a tile has, where
// operand values come from (zero outside the matrices) and where results go.  Three instances are used:
//   s^T      = W^T h^T      edge scalars from the hidden activations            (RadialWeights)
//   grad_h   = grad_s W^T   cotangent of the hidden activations                 (GradHidden)
//   grad_W^T = grad_s^T h   cotangent of the layer, per edge range of a CTA     (GradLayer, then an ordered sum)
//
// Accumulation: the tensor cores add into their float32 accumulators with truncation, so a long chain of
// products drifts (measured: 2e-5 relative after 1200 accumulation steps).  A tile of the pipeline therefore
// covers at most kGroupChunks K chunks (96 steps; kGroupChunksTma where every term has its own accumulator: 64
// steps); where a sum is longer, the epilogue warps add the finished partial tiles in float32 registers (round
// to nearest) and store once the last group has arrived (Prob::ACCUMULATE, Prob::flush).
//
// Every wait is bounded (fast::mbar_wait): on a time-out the CTA records the failure in the status word,
// stops issuing work, lets the tensor cores drain, frees its tensor memory and returns.
#pragma once
#include <cuda.h>   // CUtensorMap (the type only: the encoder is looked up at run time)

#include "fast/fast_common.cuh"
#include "umma.cuh"

namespace e3j {
namespace radial {

constexpr int kTileM = 128;      // rows of an output tile = tensor-memory lanes
constexpr int kChunkK = 32;      // k per shared-memory stage (four tcgen05.mma steps of 8)
constexpr int kStages = 3;
constexpr int kGroupChunks = 8;  // K chunks accumulated inside tensor memory before the tile is read out
constexpr int kGroupChunksTma = 16;   // the same where every term of the split has an accumulator of its own (Prob::TMA)
constexpr int kConvWarps = 8;     // converter warps
constexpr int kPrefetch = 2;      // chunks of loads in flight per converter thread (Prob::PREFETCH where given)
constexpr int kMaxResidentChunks = 4;   // K chunks of a resident A operand (Prob::A_RESIDENT): K <= 128
constexpr int kGemmThreads = (4 + kConvWarps + 1) * 32;   // epilogue, converters, tensor-core issue
constexpr int kStagesTma = 2;     // operand stages of the products whose inputs arrive as raw boxes (Prob::TMA) ...
constexpr int kRawStages = 6;     // ... and their ring of raw boxes (both even: a stage always meets the same converter group,
                                  // so every waiter sees each of its barriers' phases one after the other)
static_assert(kStagesTma % 2 == 0 && kRawStages % 2 == 0, "stages alternate between the two converter groups");
constexpr int kMaxStages = 4;     // the barrier area holds this many stage barriers of each kind

template <int N>
struct GemmSmem {
    static constexpr size_t a_bytes = (size_t)kTileM * kChunkK * 4;   // one of hi / lo
    static constexpr size_t b_bytes = (size_t)N * kChunkK * 4;
    static constexpr size_t stage_bytes = 2 * a_bytes + 2 * b_bytes;  // A_hi, A_lo, B_hi, B_lo
    static constexpr size_t off_bar = 0;       // stage_full[kMaxStages], stage_empty[kMaxStages], d_full[2], d_empty[2], drain, a_ready
    static constexpr size_t off_tmem = 8 * (2 * kMaxStages + 7);   // (... a_ready, drain of the second issuing warp)
    static constexpr size_t off_abort = off_tmem + 4;
    static constexpr size_t off_stage = 1024;
    static constexpr size_t total = off_stage + kStages * stage_bytes;
    // A operand resident (converted once per CTA): [chunks][A_hi, A_lo] first, then stages of B alone
    static constexpr size_t res_stage_bytes = 2 * b_bytes;
    static constexpr size_t res_total(int chunks) { return off_stage + (size_t)chunks * 2 * a_bytes + kStages * res_stage_bytes; }
    // raw boxes (Prob::TMA): raw_full[kRawStages], raw_empty[kRawStages] behind the other barriers; the ring starts
    // at the first 1024-byte boundary behind the operand stages (the swizzle is a function of the address)
    static constexpr size_t off_raw_bar = 128;
    static constexpr size_t raw_bytes = a_bytes + b_bytes;
    static constexpr size_t tma_total = off_stage + kStagesTma * res_stage_bytes + 1024 + kRawStages * raw_bytes;
    // tensor memory of those products: two accumulator tiles, then per stage the A operand as (hi | lo) of 32 k each
    // (an accumulator tile of those products is three: a_hi b_hi, a_hi b_lo and a_lo b_hi)
    static constexpr uint32_t tma_col_a = 6 * N, tma_cols = 512;
    static_assert(N > 64 || tma_col_a + kStagesTma * 2 * kChunkK <= tma_cols, "tensor memory");
    static_assert(off_raw_bar + 16 * kRawStages <= off_stage && off_abort + 4 <= off_raw_bar, "barrier area");
};

template <class P, class = void> struct ProbTraits {
    static constexpr bool A_RESIDENT = false;
    static constexpr int PREFETCH = kPrefetch;
};
template <class P> struct ProbTraits<P, decltype((void)P::A_RESIDENT)> {
    static constexpr bool A_RESIDENT = P::A_RESIDENT;
    static constexpr int PREFETCH = P::PREFETCH;
};

template <class P, class = void> struct TmaTraits { static constexpr bool TMA = false; };
template <class P> struct TmaTraits<P, decltype((void)P::TMA)> { static constexpr bool TMA = P::TMA; };
// (Prob::TMA: one warp more for the bulk copies and one for the second half of the tensor-core instructions)
template <class P> constexpr int gemm_threads() { return kGemmThreads + (TmaTraits<P>::TMA ? 64 : 0); }

// One box of a rank-2 tensor map into shared memory; x is the coordinate along the contiguous dimension and must
// be a multiple of four elements.  Completes on the barrier with the box's bytes, whatever part of it lay outside.
__device__ __forceinline__ void tma_load_2d(void* dst_smem, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(fast::smem_u32(dst_smem)), "l"(map), "r"(x), "r"(y), "r"(fast::smem_u32(bar)) : "memory");
}

// Converters: an operand of a stage is rows [0, ROWS) x k [0, 32).  LANE_ROWS = 8: a warp item is 8 rows x 4 k-quads
// (sources with k contiguous); LANE_ROWS = 32: 32 rows x 1 k-quad (sources with rows contiguous).  Either way 8
// consecutive lanes write 128 contiguous bytes of shared memory.  The work is two halves: all loads of a chunk go
// out first (into registers), the conversion and the stores follow one chunk later, so that the loads of chunk
// i + 1 are in flight while chunk i is converted.
template <int ROWS, int LANE_ROWS, int NW = kConvWarps>
struct OperandItems {
    static constexpr int QUADS = kChunkK / 4;
    static constexpr int LANE_QUADS = 32 / LANE_ROWS;
    static constexpr int ITEMS = (ROWS / LANE_ROWS) * (QUADS / LANE_QUADS);   // warp items of the operand
    static_assert(ROWS % LANE_ROWS == 0 && QUADS % LANE_QUADS == 0, "operand does not tile");
    static_assert(ITEMS % NW == 0, "the converter warps share the items");
    static constexpr int NI = ITEMS / NW;
    __device__ static __forceinline__ void coords(int i, int cwarp, int lane, int& row, int& k) {
        const int item = cwarp + NW * i;
        const int rg = item / (QUADS / LANE_QUADS), qg = item % (QUADS / LANE_QUADS);
        row = rg * LANE_ROWS + lane % LANE_ROWS;
        k = (qg * LANE_QUADS + lane / LANE_ROWS) * 4;
    }
    template <class Load>
    __device__ static __forceinline__ void load(float4 (&v)[NI], int cwarp, int lane, const Load& ld) {
#pragma unroll
        for (int i = 0; i < NI; ++i) {
            int row, k;
            coords(i, cwarp, lane, row, k);
            v[i] = ld(row, k);
        }
    }
    template <bool BITS = false>   // BITS: the split with integer instructions (umma::split_tf32_bits)
    __device__ static __forceinline__ void store(const float4 (&v)[NI], unsigned char* hi, unsigned char* lo, int cwarp,
                                                 int lane) {
#pragma unroll
        for (int i = 0; i < NI; ++i) {
            int row, k;
            coords(i, cwarp, lane, row, k);
            float4 h, l;
            if constexpr (BITS) umma::split_tf32_bits(v[i], h, l);
            else umma::split_tf32(v[i], h, l);
            const uint32_t off = umma::tile_offset(row, k, kChunkK);
            *reinterpret_cast<float4*>(hi + off) = h;
            *reinterpret_cast<float4*>(lo + off) = l;
        }
    }
};

template <class Prob>
__global__ void __launch_bounds__(gemm_threads<Prob>(), 1) gemm_tf32x3_kernel(const __grid_constant__ Prob prob) {
    constexpr int N = Prob::N;
    constexpr bool kTma = TmaTraits<Prob>::TMA;
    constexpr int NSTAGE = kTma ? kStagesTma : kStages;
    constexpr int DN = kTma ? 3 * N : N;   // tensor-memory columns of one accumulator tile
    using L = GemmSmem<N>;
    constexpr uint32_t kTmemCols = TmaTraits<Prob>::TMA ? L::tma_cols : 2 * N;   // two accumulator tiles (+ the A stages)
    static_assert(kTmemCols == 128 || kTmemCols == 256 || kTmemCols == 512, "tensor-memory allocation must be a power of two");
    extern __shared__ __align__(1024) unsigned char smem[];
    uint64_t* stage_full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* stage_empty = stage_full + kMaxStages;
    uint64_t* d_full = stage_empty + kMaxStages;
    uint64_t* d_empty = d_full + 2;
    uint64_t* drain = d_empty + 2;
    uint64_t* a_ready = drain + 1;
    uint64_t* drain2 = a_ready + 1;
    uint64_t* raw_full = reinterpret_cast<uint64_t*>(smem + L::off_raw_bar);
    uint64_t* raw_empty = raw_full + kRawStages;
    constexpr bool kResident = ProbTraits<Prob>::A_RESIDENT;   // A does not depend on the tile: converted once
    constexpr int kPre = ProbTraits<Prob>::PREFETCH;
    const int res_chunks = kResident ? prob.n_chunks(0) : 0;
    unsigned char* const stages = smem + L::off_stage + (size_t)res_chunks * 2 * L::a_bytes;
    static_assert(!(kResident && kTma) && NSTAGE <= kMaxStages, "one way of keeping A out of the stages at a time");
    constexpr size_t kStageBytes = (kResident || kTma) ? L::res_stage_bytes : L::stage_bytes;
    constexpr size_t kStageB = (kResident || kTma) ? 0 : 2 * L::a_bytes;   // where B_hi starts inside a stage
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::off_tmem);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        // (Prob::TMA: two issuing warps commit to stage_empty and d_full)
        for (int s = 0; s < kMaxStages; ++s) { fast::mbar_init(&stage_full[s], kTma ? kConvWarps / 2 : kConvWarps); fast::mbar_init(&stage_empty[s], kTma ? 2 : 1); }
        if constexpr (kTma)
            for (int s = 0; s < kRawStages; ++s) { fast::mbar_init(&raw_full[s], 1); fast::mbar_init(&raw_empty[s], kConvWarps / 2); }
        for (int b = 0; b < 2; ++b) { fast::mbar_init(&d_full[b], kTma ? 2 : 1); fast::mbar_init(&d_empty[b], 4); }
        fast::mbar_init(drain, 1);
        fast::mbar_init(drain2, 1);
        fast::mbar_init(a_ready, kConvWarps);
        *abort_flag = 0;
        fast::mbar_fence_init();
    }
    if (warp == 4 + kConvWarps) umma::tmem_alloc(tmem_slot, kTmemCols);
    umma::fence_before_sync();
    __syncthreads();
    umma::fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // raw boxes: behind the operand stages, at a 1024-byte boundary of the shared-memory window
    unsigned char* const raw_ring =
        smem + (((fast::smem_u32(stages + (size_t)NSTAGE * kStageBytes) + 1023u) & ~1023u) - fast::smem_u32(smem));

    const int n_tiles = prob.n_tiles();
    if (warp < 4) {
        // ------------------------------------------------ epilogue: tensor memory -> registers -> global
        float acc[Prob::ACCUMULATE ? N : 1];
#pragma unroll
        for (int i = 0; i < (Prob::ACCUMULATE ? N : 1); ++i) acc[i] = 0.f;
        for (int t = 0; t < n_tiles; ++t) {
            const int db = t & 1;
            if (!fast::mbar_wait(&d_full[db], (t >> 1) & 1, abort_flag, prob.status)) break;
            umma::fence_after_sync();
            const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(db * DN);
            const bool flush = prob.flush(t);
            if constexpr (kTma) {
                // three accumulators per tile: a_hi b_hi in columns [0, N), a_hi b_lo in [N, 2 N), a_lo b_hi behind
#pragma unroll
                for (int c0 = 0; c0 < N; c0 += 16) {
                    float v[16], u[16];
                    umma::tmem_ld16(taddr + N + c0, u);
                    umma::tmem_ld16(taddr + 2 * N + c0, v);
                    umma::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; ++i) u[i] += v[i];   // the small terms first
                    umma::tmem_ld16(taddr + c0, v);
                    umma::tmem_ld_wait();
                    if (c0 + 16 == N) {
                        umma::fence_before_sync();
                        __syncwarp();
                        if (lane == 0) fast::mbar_arrive(&d_empty[db]);
                    }
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] += u[i];
                    if constexpr (Prob::ACCUMULATE) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) { v[i] += acc[c0 + i]; acc[c0 + i] = flush ? 0.f : v[i]; }
                    }
                    if (flush) prob.store(t, warp * 32 + lane, c0, v);
                }
            } else {
#pragma unroll
            for (int c0 = 0; c0 < N; c0 += 32) {
                float v[32];
                umma::tmem_ld32(taddr + c0, v);
                umma::tmem_ld_wait();
                if (c0 + 32 == N) {   // the tile has left tensor memory: the next product may overwrite it
                    umma::fence_before_sync();
                    __syncwarp();
                    if (lane == 0) fast::mbar_arrive(&d_empty[db]);
                }
                if constexpr (Prob::ACCUMULATE) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) { v[i] += acc[c0 + i]; acc[c0 + i] = flush ? 0.f : v[i]; }
                }
                if (flush) prob.store(t, warp * 32 + lane, c0, v);
            }
            }
        }
    } else if (warp < 4 + kConvWarps) {
        // ------------------------------------------------ converters: global float32 -> (hi, lo) TF32 stages
        using OA = OperandItems<kTileM, Prob::A_LANE_ROWS>;
        using OB = OperandItems<N, Prob::B_LANE_ROWS>;
        const int cwarp = warp - 4;
        // kPrefetch chunks of loads are in flight per thread: chunk i is converted while the loads of chunks
        // i + 1 .. i + kPrefetch - 1 travel (one global-memory latency per chunk would otherwise bound the kernel)
        if constexpr (kResident) {
            for (int kc = 0; kc < res_chunks; ++kc) {
                float4 a[OA::NI];
                OA::load(a, cwarp, lane, [&](int row, int k) { return prob.load_a(0, kc, row, k); });
                unsigned char* ra = smem + L::off_stage + (size_t)kc * 2 * L::a_bytes;
                OA::store(a, ra, ra + L::a_bytes, cwarp, lane);
            }
            umma::fence_smem_to_async();
            __syncwarp();
            if (lane == 0) fast::mbar_arrive(a_ready);
        }
        if constexpr (kTma) {
            // The operands arrive as raw boxes.  A goes to tensor memory, where the tensor cores read it without
            // touching shared memory: lane m of tensor memory is row m of the tile, and a warp reaches the 32 lanes
            // of its quarter only, so a warp converts rows 32 (w % 4) ... of a chunk.  B is split into the
            // shared-memory stage as before.  The eight warps are two groups of four that take alternate chunks:
            // a chunk's way through a warp is a chain of latencies (box, tensor-memory store, proxy fence), and two
            // chunks on their way at a time hide half of it.
            using OB4 = OperandItems<N, Prob::B_LANE_ROWS, kConvWarps / 2>;
            static_assert(kConvWarps == 8, "two groups of one warp per tensor-memory quarter");
            const int grp = cwarp >> 2, qw = cwarp & 3;
            const int a_row = qw * 32 + lane;
            const uint32_t a_taddr = tmem_base + ((uint32_t)(qw * 32) << 16) + L::tma_col_a;
            int it = 0;
            bool ok = true;
            for (int t = 0; ok && t < n_tiles; ++t) {
                const int n_chunks = prob.n_chunks(t);
#pragma unroll 1
                for (int kc = 0; kc < n_chunks; ++kc, ++it) {
                    if ((it & 1) != grp) continue;
                    const int rs = it % kRawStages, s = it % NSTAGE;
                    if (!fast::mbar_wait(&raw_full[rs], (it / kRawStages) & 1, abort_flag, prob.status)) { ok = false; break; }
                    const unsigned char* ra = raw_ring + (size_t)rs * L::raw_bytes;
                    const unsigned char* rb = ra + L::a_bytes;
                    float4 a[8], b[OB4::NI];
#pragma unroll
                    for (int i = 0; i < 8; ++i) a[i] = Prob::raw_a(ra, a_row, 4 * i);
                    OB4::load(b, qw, lane, [&](int row, int k) { return Prob::raw_b(rb, row, k); });
                    if (it >= NSTAGE && !fast::mbar_wait(&stage_empty[s], ((it / NSTAGE) + 1) & 1, abort_flag, prob.status)) { ok = false; break; }
                    umma::fence_after_sync();
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        float hi[16], lo[16];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            float4 h4, l4;
                            umma::split_tf32_bits(a[4 * half + i], h4, l4);
                            hi[4 * i] = h4.x; hi[4 * i + 1] = h4.y; hi[4 * i + 2] = h4.z; hi[4 * i + 3] = h4.w;
                            lo[4 * i] = l4.x; lo[4 * i + 1] = l4.y; lo[4 * i + 2] = l4.z; lo[4 * i + 3] = l4.w;
                        }
                        umma::tmem_st16(a_taddr + (uint32_t)(s * 2 * kChunkK + 16 * half), hi);
                        umma::tmem_st16(a_taddr + (uint32_t)(s * 2 * kChunkK + kChunkK + 16 * half), lo);
                    }
                    unsigned char* st = stages + (size_t)s * kStageBytes;
                    OB4::template store<true>(b, st, st + L::b_bytes, qw, lane);
                    umma::tmem_st_wait();
                    umma::fence_before_sync();
                    umma::fence_smem_to_async();
                    __syncwarp();   // every lane's stores are out, so every lane's reads of the box have returned
                    if (lane == 0) { fast::mbar_arrive(&stage_full[s]); fast::mbar_arrive(&raw_empty[rs]); }
                }
            }
        } else {
        float4 va[kPre][kResident ? 1 : OA::NI], vb[kPre][OB::NI];
        int tf = 0, kf = 0;                      // next chunk to fetch
        int ts = 0, ks = 0;                      // next chunk to convert and store
        auto fetch = [&](float4 (&a)[kResident ? 1 : OA::NI], float4 (&b)[OB::NI]) {
            if (tf >= n_tiles) return;
            const int tt = tf, kk = kf;
            if constexpr (!kResident) OA::load(a, cwarp, lane, [&](int row, int k) { return prob.load_a(tt, kk, row, k); });
            OB::load(b, cwarp, lane, [&](int row, int k) { return prob.load_b(tt, kk, row, k); });
            if (++kf == prob.n_chunks(tf)) { kf = 0; ++tf; }
        };
#pragma unroll
        for (int u = 0; u < kPre; ++u) fetch(va[u], vb[u]);
        bool ok = true;
#pragma unroll 1
        for (int it0 = 0; ok && ts < n_tiles; it0 += kPre) {
#pragma unroll
            for (int u = 0; u < kPre; ++u) {
                if (!ok || ts >= n_tiles) break;
                const int it = it0 + u, s = it % kStages;
                if (it >= kStages && !fast::mbar_wait(&stage_empty[s], ((it / kStages) + 1) & 1, abort_flag, prob.status)) { ok = false; break; }
                unsigned char* st = stages + (size_t)s * kStageBytes;
                if constexpr (!kResident) OA::store(va[u], st, st + L::a_bytes, cwarp, lane);
                OB::store(vb[u], st + kStageB, st + kStageB + L::b_bytes, cwarp, lane);
                umma::fence_smem_to_async();
                __syncwarp();
                if (lane == 0) fast::mbar_arrive(&stage_full[s]);
                if (++ks == prob.n_chunks(ts)) { ks = 0; ++ts; }
                fetch(va[u], vb[u]);             // refill this register set with the chunk kPre ahead
            }
        }
        }
    } else if (warp == 4 + kConvWarps || (kTma && warp == 4 + kConvWarps + 2)) {
        // ------------------------------------------------ tensor-core issue (one lane; Prob::TMA: of two warps)
        const bool second = warp != 4 + kConvWarps;
        constexpr uint32_t idesc = umma::idesc_tf32(kTileM, N);
        const uint32_t sbo = umma::sbo_bytes(kChunkK);
        int it = 0;
        bool ok = true;
        if (kResident && n_tiles > 0 && !fast::mbar_wait(a_ready, 0, abort_flag, prob.status)) ok = false;
        for (int t = 0; ok && t < n_tiles; ++t) {
            const int db = t & 1;
            const int n_chunks = prob.n_chunks(t);
            if (t >= 2 && !fast::mbar_wait(&d_empty[db], ((t >> 1) + 1) & 1, abort_flag, prob.status)) break;
            for (int kc = 0; kc < n_chunks; ++kc, ++it) {
                const int s = it % NSTAGE;
                if (!fast::mbar_wait(&stage_full[s], (it / NSTAGE) & 1, abort_flag, prob.status)) { ok = false; break; }
                umma::fence_after_sync();
                if (lane == 0) {
                    const uint32_t st = umma::smem_addr(stages + (size_t)s * kStageBytes);
                    const uint32_t b_hi = st + (uint32_t)kStageB, b_lo = b_hi + (uint32_t)L::b_bytes;
                    const uint32_t d = tmem_base + (uint32_t)(db * DN);
                    // small terms first: a_lo b_hi, a_hi b_lo, then a_hi b_hi
                    const uint32_t pb[3] = {b_hi, b_lo, b_hi};
                    if constexpr (kTma) {
                        // A in tensor memory: columns (hi | lo) of the stage.  The issuing thread is what bounds
                        // these products (an instruction of N = 64 is over before the next one is out), so the
                        // passes are folded and shared between two warps.  B_hi and B_lo lie behind each other
                        // in the stage and serve as one operand of 2 N rows: the first warp issues
                        // a_hi [b_hi | b_lo] into the tile's first two accumulators, the second a_lo b_hi into
                        // the third (accumulators of their own, so the order of the sums does not depend on
                        // which warp is ahead); the epilogue adds the three.
                        const uint32_t a_hi = tmem_base + L::tma_col_a + (uint32_t)(s * 2 * kChunkK), a_lo = a_hi + kChunkK;
                        constexpr uint32_t idesc2 = umma::idesc_tf32(kTileM, 2 * N);
                        if (!second) {
#pragma unroll
                            for (int ks = 0; ks < kChunkK / 8; ++ks)
                                umma::mma_tf32_ts(d, a_hi + ks * 8, umma::make_desc(b_hi + ks * 2 * umma::kLbo, umma::kLbo, sbo), idesc2,
                                                  (kc > 0 || ks > 0) ? 1u : 0u);
                        } else {
#pragma unroll
                            for (int ks = 0; ks < kChunkK / 8; ++ks)
                                umma::mma_tf32_ts(d + 2 * N, a_lo + ks * 8, umma::make_desc(b_hi + ks * 2 * umma::kLbo, umma::kLbo, sbo), idesc,
                                                  (kc > 0 || ks > 0) ? 1u : 0u);
                        }
                    } else {
                        const uint32_t a_hi = kResident ? umma::smem_addr(smem + L::off_stage + (size_t)kc * 2 * L::a_bytes) : st;
                        const uint32_t a_lo = a_hi + (uint32_t)L::a_bytes;
                        const uint32_t pa[3] = {a_lo, a_hi, a_hi};
#pragma unroll
                        for (int pass = 0; pass < 3; ++pass)
#pragma unroll
                            for (int ks = 0; ks < kChunkK / 8; ++ks)
                                umma::mma_tf32(d, umma::make_desc(pa[pass] + ks * 2 * umma::kLbo, umma::kLbo, sbo),
                                               umma::make_desc(pb[pass] + ks * 2 * umma::kLbo, umma::kLbo, sbo), idesc,
                                               (kc > 0 || pass > 0 || ks > 0) ? 1u : 0u);
                    }
                    umma::commit(&stage_empty[s]);                       // the stage may be refilled
                    if (kc == n_chunks - 1) umma::commit(&d_full[db]);   // the tile is complete
                }
                __syncwarp();
            }
        }
        // abort path only: let the products still in flight finish before tensor memory is freed
        if (*abort_flag) {
            uint64_t* const mine = second ? drain2 : drain;
            if (lane == 0) umma::commit(mine);
            __syncwarp();
#pragma unroll 1
            for (uint32_t spin = 0; spin < fast::kSpinLimit; ++spin)
                if (fast::mbar_try_wait(mine, 0)) break;
        }
    } else {
        // ------------------------------------------------ raw boxes (Prob::TMA): tiled bulk copies, one lane
        if constexpr (kTma) {
            int it = 0;
            bool ok = true;
            for (int t = 0; ok && t < n_tiles; ++t) {
                const int n_chunks = prob.n_chunks(t);
#pragma unroll 1
                for (int kc = 0; kc < n_chunks; ++kc, ++it) {
                    const int rs = it % kRawStages;
                    if (it >= kRawStages && !fast::mbar_wait(&raw_empty[rs], ((it / kRawStages) + 1) & 1, abort_flag, prob.status)) { ok = false; break; }
                    if (lane == 0) {
                        unsigned char* ra = raw_ring + (size_t)rs * L::raw_bytes;
                        int x, y;
                        fast::mbar_arrive_expect_tx(&raw_full[rs], (uint32_t)L::raw_bytes);
                        prob.box_a(t, kc, x, y);
                        tma_load_2d(ra, &prob.map_a, x, y, &raw_full[rs]);
                        prob.box_b(t, kc, x, y);
                        tma_load_2d(ra + L::a_bytes, &prob.map_b, x, y, &raw_full[rs]);
                    }
                    __syncwarp();
                }
            }
            // abort path only: the copies still in flight must land before the CTA gives its shared memory back
            if (*abort_flag) {
                for (int j = max(0, it - kRawStages); j < it; ++j) {
#pragma unroll 1
                    for (uint32_t spin = 0; spin < fast::kSpinLimit; ++spin)
                        if (fast::mbar_try_wait(&raw_full[j % kRawStages], (j / kRawStages) & 1)) break;
                }
            }
        }
    }
    umma::fence_before_sync();
    __syncthreads();
    if (warp == 4 + kConvWarps) umma::tmem_dealloc(tmem_base, kTmemCols);
}

// Reads of a raw box by the converters.  Rows of 128 bytes under the 128-byte swizzle: the 16-byte piece j of
// row r lies at piece j ^ (r % 8) of that row (the box starts at a 1024-byte boundary).
__device__ __forceinline__ float4 raw_swizzled(const unsigned char* box, int row, int k) {
    return *reinterpret_cast<const float4*>(box + row * 128 + ((((k >> 2) ^ row) & 7) << 4));
}
// Plain boxes of `pitch` floats per row, read across the rows: element (k + i, row) for i < 4.
__device__ __forceinline__ float4 raw_transposed(const unsigned char* box, int pitch, int row, int k) {
    const float* b = reinterpret_cast<const float*>(box) + k * pitch + row;
    return make_float4(b[0], b[pitch], b[2 * pitch], b[3 * pitch]);
}

// ------------------------------------------------------------------------------------------------ problems
// s[e, c] = sum_j h[e, j] W[j, c]: tile (column block cb of 128 c) x (128 edges); m = c, n = edge, k = j.
struct RadialWeights {
    static constexpr int N = 128, A_LANE_ROWS = 32, B_LANE_ROWS = 8;
    static constexpr bool ACCUMULATE = false;   // k = hidden is short: one chain per tile
    static constexpr bool A_RESIDENT = true;    // the CTA's block of W^T serves all of its tiles
    static constexpr int PREFETCH = 4;          // two tiles of h in flight per converter thread
    __device__ __forceinline__ bool flush(int) const { return true; }
    const float* h; const float* W; float* s;
    int64_t n_edges, chunk;   // chunk: edges per CTA row of the grid (multiple of 128)
    int H, C;
    int32_t* status;
    __device__ __forceinline__ int64_t e_begin() const { return min(n_edges, (int64_t)blockIdx.y * chunk); }
    __device__ __forceinline__ int n_tiles() const {
        const int64_t e0 = e_begin(), e1 = min(n_edges, e0 + chunk);
        return (int)((e1 - e0 + 127) / 128);
    }
    __device__ __forceinline__ int n_chunks(int) const { return (H + kChunkK - 1) / kChunkK; }
    __device__ __forceinline__ float4 load_a(int, int kc, int row, int k) const {   // W^T: row = c, k = j
        const int c = blockIdx.x * 128 + row, j = kc * kChunkK + k;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < C) {
            if (j + 0 < H) v.x = W[(size_t)(j + 0) * C + c];
            if (j + 1 < H) v.y = W[(size_t)(j + 1) * C + c];
            if (j + 2 < H) v.z = W[(size_t)(j + 2) * C + c];
            if (j + 3 < H) v.w = W[(size_t)(j + 3) * C + c];
        }
        return v;
    }
    __device__ __forceinline__ float4 load_b(int t, int kc, int row, int k) const {   // h: row = edge, k = j
        const int64_t e = e_begin() + (int64_t)t * 128 + row;
        const int j = kc * kChunkK + k;
        if (e >= n_edges || e >= e_begin() + chunk || j >= H) return make_float4(0.f, 0.f, 0.f, 0.f);
        return *reinterpret_cast<const float4*>(h + (size_t)e * H + j);   // H % 4 == 0
    }
    template <int W>
    __device__ __forceinline__ void store(int t, int m, int n0, const float (&v)[W]) const {
        const int c = blockIdx.x * 128 + m;
        if (c >= C) return;
        const int64_t e0 = e_begin() + (int64_t)t * 128 + n0;
        const int64_t e_end = min(n_edges, e_begin() + chunk);
        float* dst = s + (size_t)e0 * C + c;   // lanes: consecutive c; one row of s further per value
        if (e0 + W <= e_end) {                 // whole piece inside the range: no per-store test
#pragma unroll
            for (int i = 0; i < W; ++i) dst[(size_t)i * C] = v[i];
        } else {
#pragma unroll
            for (int i = 0; i < W; ++i)
                if (e0 + i < e_end) dst[(size_t)i * C] = v[i];
        }
    }
};

// the same product for hidden widths beyond kMaxResidentChunks * 32: both operands converted per tile
struct RadialWeightsWide : RadialWeights {
    static constexpr bool A_RESIDENT = false;
    static constexpr int PREFETCH = kPrefetch;
};

// grad_h[e, j] = sum_c grad_s[e, c] W[j, c]: tile = 128 edges x (64 j, block blockIdx.y); m = edge, n = j, k = c.
struct GradHidden {
    static constexpr int N = 64, A_LANE_ROWS = 8, B_LANE_ROWS = 8;
    static constexpr bool ACCUMULATE = true;
    static constexpr bool TMA = true;
    alignas(64) CUtensorMap map_a, map_b;   // grad_s [n_edges][C], W [H][C]
    const float* gs; const float* W; float* gh;
    int64_t n_edges, chunk;   // chunk: edges per CTA (multiple of 128)
    int H, C;
    int gc;                   // K chunks summed inside tensor memory before a tile is read out (see the head of the file)
    int32_t* status;
    // pipeline tile t = (edge tile t / groups, group t % groups of gc chunks of c)
    __device__ __forceinline__ int total_chunks() const { return (C + kChunkK - 1) / kChunkK; }
    __device__ __forceinline__ int groups() const { return (total_chunks() + gc - 1) / gc; }
    __device__ __forceinline__ int64_t e_begin() const { return min(n_edges, (int64_t)blockIdx.x * chunk); }
    __device__ __forceinline__ int n_tiles() const {
        const int64_t e0 = e_begin(), e1 = min(n_edges, e0 + chunk);
        return (int)((e1 - e0 + 127) / 128) * groups();
    }
    __device__ __forceinline__ int n_chunks(int t) const {
        return min(gc, total_chunks() - (t % groups()) * gc);
    }
    __device__ __forceinline__ bool flush(int t) const { return t % groups() == groups() - 1; }
    // operands: boxes of 32 c (128 edges of grad_s | 64 rows of W), 128-byte swizzle
    __device__ __forceinline__ int first_c(int t, int kc) const { return ((t % groups()) * gc + kc) * kChunkK; }
    __device__ __forceinline__ void box_a(int t, int kc, int& x, int& y) const {
        x = first_c(t, kc); y = (int)(e_begin() + (int64_t)(t / groups()) * 128);
    }
    __device__ __forceinline__ void box_b(int t, int kc, int& x, int& y) const { x = first_c(t, kc); y = blockIdx.y * 64; }
    __device__ static __forceinline__ float4 raw_a(const unsigned char* box, int row, int k) { return raw_swizzled(box, row, k); }
    __device__ static __forceinline__ float4 raw_b(const unsigned char* box, int row, int k) { return raw_swizzled(box, row, k); }
    template <int W>
    __device__ __forceinline__ void store(int t, int m, int n0, const float (&v)[W]) const {
        const int64_t e = e_begin() + (int64_t)(t / groups()) * 128 + m;
        if (e >= n_edges || e >= e_begin() + chunk) return;
        const int j0 = blockIdx.y * 64 + n0;
#pragma unroll
        for (int i = 0; i < W; i += 4)
            if (j0 + i < H)   // H % 4 == 0
                *reinterpret_cast<float4*>(gh + (size_t)e * H + j0 + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
    }
};

// partial[r, j, c] = sum over the edges of range r of h[e, j] grad_s[e, c]: one tile per CTA,
// m = c (column block of 128), n = j (block blockIdx.z of 64), k = edge.  grad_W = sum_r partial[r] in range
// order (layer_sum_kernel).
struct GradLayer {
    static constexpr int N = 64, A_LANE_ROWS = 32, B_LANE_ROWS = 32;
    static constexpr bool ACCUMULATE = true;
    static constexpr bool TMA = true;
    alignas(64) CUtensorMap map_a, map_b;   // grad_s [n_edges][C], h [n_edges][H]
    const float* gs; const float* h; float* partial;
    int64_t n_edges, chunk;   // chunk: edges per range (multiple of 32)
    int H, C;
    int gc;                   // K chunks summed inside tensor memory before a tile is read out
    int32_t* status;
    __device__ __forceinline__ int64_t e_begin() const { return min(n_edges, (int64_t)blockIdx.y * chunk); }
    // pipeline tile t = group t of gc chunks of the range's edges; one output tile per CTA
    __device__ __forceinline__ int total_chunks() const {
        const int64_t e0 = e_begin(), e1 = min(n_edges, e0 + chunk);
        return (int)max((int64_t)1, (e1 - e0 + kChunkK - 1) / kChunkK);   // an empty range still writes a zero tile
    }
    __device__ __forceinline__ int n_tiles() const { return (total_chunks() + gc - 1) / gc; }
    __device__ __forceinline__ int n_chunks(int t) const { return min(gc, total_chunks() - t * gc); }
    __device__ __forceinline__ bool flush(int t) const { return t == n_tiles() - 1; }
    // operands: boxes of 32 edges (128 c of grad_s | 64 j of h), read across the rows
    __device__ __forceinline__ int first_e(int t, int kc) const { return (int)(e_begin() + (int64_t)(t * gc + kc) * kChunkK); }
    __device__ __forceinline__ void box_a(int t, int kc, int& x, int& y) const { x = blockIdx.x * 128; y = first_e(t, kc); }
    __device__ __forceinline__ void box_b(int t, int kc, int& x, int& y) const { x = blockIdx.z * 64; y = first_e(t, kc); }
    __device__ static __forceinline__ float4 raw_a(const unsigned char* box, int row, int k) { return raw_transposed(box, 128, row, k); }
    __device__ static __forceinline__ float4 raw_b(const unsigned char* box, int row, int k) { return raw_transposed(box, 64, row, k); }
    template <int W>
    __device__ __forceinline__ void store(int, int m, int n0, const float (&v)[W]) const {
        const int c = blockIdx.x * 128 + m;
        if (c >= C) return;
        const int j0 = blockIdx.z * 64 + n0;
        float* dst = partial + (size_t)blockIdx.y * H * C + (size_t)j0 * C + c;   // lanes: consecutive c
        if (j0 + W <= H) {
#pragma unroll
            for (int i = 0; i < W; ++i) dst[(size_t)i * C] = v[i];
        } else {
#pragma unroll
            for (int i = 0; i < W; ++i)
                if (j0 + i < H) dst[(size_t)i * C] = v[i];
        }
    }
};

// grad_W[j, c] = sum_r partial[r, j, c], r ascending.
__global__ void layer_sum_kernel(int n_ranges, int64_t n_elems, const float* __restrict__ partial, float* __restrict__ grad_W);

}  // namespace radial
}  // namespace e3j
