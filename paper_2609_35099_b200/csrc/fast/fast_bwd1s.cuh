// Scheduled edge-wise backward: fast_bwd1.cuh's sweep over a processing order built once per neighbour list
// (csrc/bwd_schedule.hpp), in which the edges of one sender into neighbouring receivers follow one another in one
// consumer warp.  The warp keeps the sum of their grad_x shares in registers and writes one row per run instead of
// one per edge; the sender sum reads those rows, contiguous per sender, in a fixed order.
//
// Differences from the plain edge-wise kernel:
//   * a tile's T slots are any edges of the CTA's range (the schedule names them), so every slot has its own bulk
//     copies of the weight row and the sender row, and its harmonics are gathered by edge id;
//   * the grad_out rows of three receivers are resident; the schedule says with which tile a row is loaded (never
//     while a tile in flight may still read the slot's previous occupant);
//   * tile records (16 bytes per slot + 16 per tile) arrive in windows of WT tiles through 16-byte asynchronous
//     copies, two windows ahead; the harmonics of a window are fetched once its records are in shared memory,
//     one window ahead.
// Graph calls only (no padded lists, no standalone tensor product, no double backward), one warp per edge.
#pragma once
#include "../bwd_schedule.hpp"
#include "fast_bwd1.cuh"

namespace e3j {
namespace fast {

constexpr int kStatusBadSchedule = 3;   // the schedule does not belong to this kernel / grid

struct SchedParams {
    const float* x; const float* sh; const float* w; const float* grad_out;
    float* grad_sh; float* grad_w;
    float* dx_rows;           // scratch [n_rows][d][N_q]
    const int32_t* sched;     // words of the schedule
    int32_t* status;
};

__device__ __forceinline__ void cp_async16(void* dst_smem, const void* src_gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst_smem)), "l"(src_gmem) : "memory");
}

template <class S>
struct Bwd1sSmem {
    static constexpr int T = S::ET, NS = kSchedStages, NSLOT = kSchedSlots;
    static constexpr int VW = S::EV;
    using Vec = typename VecOf<VW>::type;
    static_assert(S::NQ == 32 * VW, "one warp per edge");
    static constexpr int S_EDGE = S::P * S::NQ;
    static constexpr int X_EDGE = S::DIN * S::NQ;
    static constexpr int DM_ROW = S::D * S::NQ;
    static constexpr int REC = T + 1;            // 16-byte records per tile
    static constexpr int WT = 32 / REC;          // tiles per window of records (one warp-wide copy)
    static_assert(WT >= NS, "a window must outlast the tiles in flight");
    static constexpr size_t up(size_t v, size_t a) { return (v + a - 1) / a * a; }
    static constexpr size_t off_bar = 0;                                    // full[NS], empty[NS]
    static constexpr size_t off_abort = off_bar + 16 * NS;
    static constexpr size_t off_meta = up(off_abort + 4, 16);               // int4[NS][T]: edge, row, -, grad_out slot
    static constexpr size_t off_info = off_meta + 16 * NS * T;              // int4[3][32]: windows of tile records
    static constexpr size_t off_y = off_info + 16 * 3 * 32;                 // float[2][WT * T][DSH]
    static constexpr size_t off_dm = up(off_y + 4 * 2 * WT * T * S::DSH, 128);   // float[NSLOT][D][NQ]
    static constexpr size_t off_stage = up(off_dm + 4 * (size_t)NSLOT * DM_ROW, 128);
    static constexpr size_t st_s = 0;
    static constexpr size_t st_x = st_s + 4 * (size_t)T * S_EDGE;
    static constexpr size_t st_A = st_x + 4 * (size_t)T * X_EDGE;
    static constexpr size_t stage_bytes = up(st_A + 4 * (size_t)T * S::B_APAD, 128);
    static constexpr size_t total = off_stage + NS * stage_bytes;
};

// ------------------------------------------------------------------------ consumer: column `warp` of every tile
template <class S>
__device__ __forceinline__ void bwd1s_consumer(const SchedParams& p, unsigned char* smem, const int warp, const int lane,
                                               const int n_tiles) {
    using L = Bwd1sSmem<S>;
    using Vec = typename L::Vec;
    constexpr int NS = L::NS, VW = L::VW, NQV = S::NQ / VW;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* empty = full + NS;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    int stage = 0, phase = 0;
    bool open = false;     // a run is in progress: acc holds the sum of its shares so far
    Vec acc[S::DIN];
#pragma unroll 1
    for (int t = 0; t < n_tiles; ++t) {
        if (!mbar_wait(&full[stage], phase, abort_flag, p.status)) break;
        const int4 m = reinterpret_cast<const int4*>(smem + L::off_meta)[stage * L::T + warp];
        if (m.x >= 0) {
            const unsigned char* st = smem + L::off_stage + stage * (int)L::stage_bytes;
            const int64_t e = m.x;
            const Vec* xs = reinterpret_cast<const Vec*>(st + L::st_x) + warp * (L::X_EDGE / VW) + lane;
            const Vec* ss = reinterpret_cast<const Vec*>(st + L::st_s) + warp * (L::S_EDGE / VW) + lane;
            const float* As = reinterpret_cast<const float*>(st + L::st_A) + warp * S::B_APAD;
            const Vec* dms = reinterpret_cast<const Vec*>(smem + L::off_dm + (size_t)m.w * 4 * L::DM_ROW) + lane;
            Vec dxp[S::DIN];
            float dyl[16];
            Vec* gw = reinterpret_cast<Vec*>(p.grad_w + (size_t)e * L::S_EDGE) + lane;
            S::bwd_edge_all(dms, xs, ss, As, dxp, dyl, gw);
#pragma unroll
            for (int i = 0; i < S::DIN; ++i) acc[i] = open ? vadd(acc[i], dxp[i]) : dxp[i];
            open = m.y < 0;
            if (!open) {   // the run ends here: its row
                Vec* dxo = reinterpret_cast<Vec*>(p.dx_rows + (size_t)m.y * L::X_EDGE) + lane;
#pragma unroll
                for (int i = 0; i < S::DIN; ++i) dxo[i * NQV] = acc[i];
            }
            const float dy_tot = reduce16_over_lanes(dyl, lane);
            const int idx = ((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1);
            if ((lane & 1) == 0 && idx < S::DSH) p.grad_sh[(size_t)e * S::DSH + idx] = dy_tot;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[stage]);
        if (++stage == NS) { stage = 0; phase ^= 1; }
    }
}

// ------------------------------------------------------------------------ producer
template <class S>
__device__ __forceinline__ void bwd1s_producer(const SchedParams& p, unsigned char* smem, const int lane,
                                               const int4* __restrict__ recs, const int n_tiles) {
    using L = Bwd1sSmem<S>;
    using Tab = BwdTab<S>;
    constexpr int T = L::T, NS = L::NS, WT = L::WT, REC = L::REC, DSH = S::DSH;
    constexpr int NA = (Tab::APAD + 31) / 32;
    static_assert(T <= 28 && L::NSLOT <= 4, "lanes 28.. of the producer issue the grad_out row loads");
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* empty = full + NS;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    int4* info = reinterpret_cast<int4*>(smem + L::off_info);
    float* y_ring = reinterpret_cast<float*>(smem + L::off_y);
    const int n_win = (n_tiles + WT - 1) / WT;

    ASlot tab[NA];   // this lane's A slots (lane, lane + 32, ...)
#pragma unroll
    for (int i = 0; i < NA; ++i) {
        const int slot = lane + 32 * i;
        ASlot a{0.f, 0.f, 0, 0};
        if (slot < Tab::APAD) {
            const PairRec pr = Tab::pair_rec(slot);
            if (pr.count > 0) { a.c0 = Tab::rec_val(pr.start); a.i2_0 = Tab::rec_i2(pr.start); }
            if (pr.count > 1) { a.c1 = Tab::rec_val(pr.start + 1); a.i2_1 = Tab::rec_i2(pr.start + 1); }
        }
        tab[i] = a;
    }

    // one copy group per call, also when there is nothing to copy: the waits below count groups
    auto issue_info = [&](const int w) {
        if (w < n_win) {
            const int count = min(WT, n_tiles - w * WT) * REC;
            if (lane < count) cp_async16(&info[(w % 3) * 32 + lane], recs + (size_t)w * WT * REC + lane);
        }
        cp_async_commit();
    };
    auto issue_y = [&](const int w) {   // the records of window w are in shared memory
        if (w < n_win && lane < min(WT, n_tiles - w * WT) * T) {
            const int i = lane / T, j = lane - i * T;
            const int e = info[(w % 3) * 32 + i * REC + j].x;
            if (e >= 0) {
                float* dst = y_ring + (size_t)((w & 1) * WT * T + lane) * DSH;
                const float* src = p.sh + (size_t)e * DSH;
                if constexpr (DSH % 4 == 0) {
#pragma unroll
                    for (int k = 0; k < DSH; k += 4) cp_async16(dst + k, src + k);
                } else {
#pragma unroll
                    for (int k = 0; k < DSH; ++k) cp_async4(dst + k, src + k);
                }
            }
        }
        cp_async_commit();
    };
    issue_info(0);
    issue_info(1);
    cp_async_wait<1>();   // records of window 0
    __syncwarp();
    issue_y(0);

    int stage = 0, phase = 0, armed = 0;
#pragma unroll 1
    for (int t = 0; t < n_tiles; ++t) {
        const int w = t / WT, i = t - w * WT;
        if (i == 0) {
            issue_info(w + 2);
            cp_async_wait<1>();   // all but the newest group: the records of window w + 1 and the harmonics of window w
            __syncwarp();
            issue_y(w + 1);
        }
        // phase of `empty` that ends the previous use of this ring slot (and of the grad_out slots loaded below)
        if (t >= NS && !mbar_wait(&empty[stage], phase ^ 1, abort_flag, p.status)) break;
        const int4* rec = info + (w % 3) * 32 + i * REC;
        int4 r = make_int4(-1, -1, -1, 0);
        if (lane < T) r = rec[lane];
        const bool valid = r.x >= 0;
        const unsigned vmask = __ballot_sync(0xffffffffu, valid);
        int load_r = -1;
        if (lane >= 28 && lane < 28 + L::NSLOT) {
            const int4 lr = rec[T];
            load_r = lane == 28 ? lr.x : lane == 29 ? lr.y : lr.z;
        }
        const unsigned lmask = __ballot_sync(0xffffffffu, load_r >= 0);
        unsigned char* st = smem + L::off_stage + stage * (int)L::stage_bytes;
        if (lane < T) reinterpret_cast<int4*>(smem + L::off_meta)[stage * T + lane] = make_int4(r.x, r.z, 0, r.w);
        if (lane == 0)   // arrival and byte count in one step: the phase cannot complete before the bytes are expected
            mbar_arrive_expect_tx(&full[stage], (uint32_t)__popc(vmask) * 4u * (L::S_EDGE + L::X_EDGE) +
                                                    (uint32_t)__popc(lmask) * 4u * L::DM_ROW);
        if (valid) {
            bulk_g2s(st + L::st_s + (size_t)lane * 4 * L::S_EDGE, p.w + (size_t)r.x * L::S_EDGE, 4u * L::S_EDGE, &full[stage]);
            bulk_g2s(st + L::st_x + (size_t)lane * 4 * L::X_EDGE, p.x + (size_t)r.y * L::X_EDGE, 4u * L::X_EDGE, &full[stage]);
        }
        if (load_r >= 0)
            bulk_g2s(smem + L::off_dm + (size_t)(lane - 28) * 4 * L::DM_ROW, p.grad_out + (size_t)load_r * L::DM_ROW,
                     4u * L::DM_ROW, &full[stage]);
        armed = t + 1;
        // A[slot][entry] = sum over the entry's records of c * y[i2]; all loads before the first store
        // (entries of empty slots are computed from stale data and never read)
        {
            float* A_t = reinterpret_cast<float*>(st + L::st_A);
            const float* yw = y_ring + (size_t)((w & 1) * WT * T + i * T) * DSH;
            float a_val[NA][T];
#pragma unroll
            for (int k = 0; k < NA; ++k)
#pragma unroll
                for (int e_i = 0; e_i < T; ++e_i) {
                    const float* ye = yw + e_i * DSH;
                    a_val[k][e_i] = fmaf(tab[k].c1, ye[tab[k].i2_1], tab[k].c0 * ye[tab[k].i2_0]);
                }
#pragma unroll
            for (int k = 0; k < NA; ++k) {
                const int slot = lane + 32 * k;
                if (slot < Tab::APAD) {
#pragma unroll
                    for (int e_i = 0; e_i < T; ++e_i) A_t[e_i * Tab::APAD + slot] = a_val[k][e_i];
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&full[stage]);   // the A entries and the tile's slot records are in place
        if (++stage == NS) { stage = 0; phase ^= 1; }
    }
    cp_async_wait<0>();
    if (*abort_flag) drain_copies<L>(smem, armed);
}

template <class S>
__global__ void __launch_bounds__((S::ET + 1) * 32, 1) fast_bwd1s_kernel(const SchedParams p) {
    using L = Bwd1sSmem<S>;
    constexpr int T = L::T, NS = L::NS;
    static_assert(S::B_NREC <= 2, "an A slot holds at most two records");
    static_assert(S::DSH <= 16, "harmonics beyond l = 3 need a wider reduction");
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* empty = full + NS;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const int32_t* hdr = p.sched;
    if (hdr[0] != kSchedMagic || hdr[1] != T || hdr[2] != L::NSLOT || hdr[3] != (int)gridDim.x) {
        if (threadIdx.x == 0) atomicCAS(p.status, 0, kStatusBadSchedule);
        return;
    }
    const int32_t* tile_ptr = hdr + hdr[8];
    const int t0 = tile_ptr[blockIdx.x], n_tiles = tile_ptr[blockIdx.x + 1] - t0;
    if (n_tiles <= 0) return;
    const int4* recs = reinterpret_cast<const int4*>(hdr + hdr[10]) + (size_t)t0 * L::REC;

    if (threadIdx.x == 0) {
        // full: the producer's arrival with the copies' byte count and its arrival after the tables;
        // empty: the T warps that work on the slot
        for (int s = 0; s < NS; ++s) { mbar_init(&full[s], 2); mbar_init(&empty[s], T); }
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    if (warp == T) bwd1s_producer<S>(p, smem, lane, recs, n_tiles);
    else bwd1s_consumer<S>(p, smem, warp, lane, n_tiles);
}

// grad_x[a] = sum of the rows of a's runs, in processing order (contiguous: row_ptr[a] .. row_ptr[a + 1])
__global__ void bwd_rows_reduce_kernel(int64_t n_nodes, int row_f4, const float4* __restrict__ dx_rows,
                                       const int32_t* __restrict__ row_ptr, float4* __restrict__ grad_x);

template <class S>
int launch_bwd_sched(const ConvArgs& a, const int32_t* sched) {
    using L = Bwd1sSmem<S>;
    static_assert(L::total + 1024 <= 228 * 1024, "scheduled backward ring does not fit in shared memory");
    if (a.workspace_bytes < bwd_scratch_bytes<S>(a.n_nodes, a.n_edges)) return E3J_ERR_WORKSPACE;   // rows <= edges
    const int n_cta = sm_count();
    SchedParams p{};
    p.x = a.x; p.sh = a.sh; p.w = a.w; p.grad_out = a.grad_out; p.grad_sh = a.grad_sh; p.grad_w = a.grad_w;
    p.dx_rows = reinterpret_cast<float*>(a.workspace);
    p.sched = sched; p.status = a.status;
    static thread_local int attr_dev = -1;
    int dev = 0;
    E3J_CUDA_TRY(cudaGetDevice(&dev));
    if (attr_dev != dev) {
        E3J_CUDA_TRY(cudaFuncSetAttribute(fast_bwd1s_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::total));
        attr_dev = dev;
    }
    fast_bwd1s_kernel<S><<<n_cta, (L::T + 1) * 32, L::total, a.stream>>>(p);
    if (int s = after_launch()) return s;
    const int32_t* row_ptr = sched + 16 + n_cta + 1;   // header, tile_ptr[n_cta + 1], then row_ptr (bwd_schedule.hpp)
    const int64_t blocks = std::min<int64_t>(a.n_nodes, (int64_t)1 << 30);
    return launch_dependent(bwd_rows_reduce_kernel, dim3((int)blocks), dim3(S::DIN * S::NQ / 4), 0, a.stream, a.n_nodes, S::DIN * S::NQ / 4,
        reinterpret_cast<const float4*>(p.dx_rows), row_ptr, reinterpret_cast<float4*>(a.grad_x));
}

}  // namespace fast
}  // namespace e3j
