// Building blocks of the signature-specialised kernels (sm_100a).
//
// Data movement: edge-local operands (weights, harmonics) stream through a ring of
// shared-memory stages filled by bulk asynchronous copies (cp.async.bulk, completion
// counted on an mbarrier); sender rows are gathered into the same stage by one bulk
// copy per edge.  One producer warp issues the copies, the consumer warps wait on the
// stage's "full" barrier and hand the stage back through its "empty" barrier.
// Plain bulk copies only (no tensor maps, nothing shared across a cluster): every copy is a contiguous,
// 16-byte aligned range.
//
// Every wait is bounded: after kSpinLimit failed polls a warp records an error in the
// status word, and the CTA drains and returns instead of spinning forever.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

namespace e3j {
namespace fast {

constexpr uint32_t kSpinLimit = 1u << 22;  // polls of mbarrier.try_wait before giving up
constexpr int kStatusTimeout = 1;          // value stored in the device status word

// First statement of a kernel that is launched with launch_dependent (common.cuh): holds the kernel until the
// one before it on the stream has finished and its writes are visible; a no-op under an ordinary launch.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---------------------------------------------------------------- channel vectors
// A lane owns V consecutive channels (float2 or float4): one 8- or 16-byte shared-memory
// load feeds V FMAs.
__device__ __forceinline__ float4 vmul(const float4 a, const float4 b) {
    return make_float4(a.x * b.x, a.y * b.y, a.z * b.z, a.w * b.w);
}
__device__ __forceinline__ float2 vmul(const float2 a, const float2 b) { return make_float2(a.x * b.x, a.y * b.y); }
__device__ __forceinline__ void vfma(float4& acc, const float a, const float4 b) {
    acc.x = fmaf(a, b.x, acc.x); acc.y = fmaf(a, b.y, acc.y); acc.z = fmaf(a, b.z, acc.z); acc.w = fmaf(a, b.w, acc.w);
}
__device__ __forceinline__ void vfma(float2& acc, const float a, const float2 b) {
    acc.x = fmaf(a, b.x, acc.x); acc.y = fmaf(a, b.y, acc.y);
}
__device__ __forceinline__ void vfma(float4& acc, const float4 a, const float4 b) {
    acc.x = fmaf(a.x, b.x, acc.x); acc.y = fmaf(a.y, b.y, acc.y); acc.z = fmaf(a.z, b.z, acc.z); acc.w = fmaf(a.w, b.w, acc.w);
}
__device__ __forceinline__ void vfma(float2& acc, const float2 a, const float2 b) {
    acc.x = fmaf(a.x, b.x, acc.x); acc.y = fmaf(a.y, b.y, acc.y);
}
// Two channels per instruction: the packed single-precision multiply / fused multiply-add of sm_100 (one issue
// slot for two IEEE operations, bit-identical to the scalar forms).
__device__ __forceinline__ float2 pmul(const float2 a, const float2 b) { return __fmul2_rn(a, b); }
__device__ __forceinline__ float4 pmul(const float4 a, const float4 b) {
    const float2 lo = __fmul2_rn(make_float2(a.x, a.y), make_float2(b.x, b.y));
    const float2 hi = __fmul2_rn(make_float2(a.z, a.w), make_float2(b.z, b.w));
    return make_float4(lo.x, lo.y, hi.x, hi.y);
}
__device__ __forceinline__ void pfma(float2& acc, const float2 a, const float2 b) { acc = __ffma2_rn(a, b, acc); }
__device__ __forceinline__ void pfma(float2& acc, const float a, const float2 b) { acc = __ffma2_rn(make_float2(a, a), b, acc); }
__device__ __forceinline__ void pfma(float4& acc, const float4 a, const float4 b) {
    const float2 lo = __ffma2_rn(make_float2(a.x, a.y), make_float2(b.x, b.y), make_float2(acc.x, acc.y));
    const float2 hi = __ffma2_rn(make_float2(a.z, a.w), make_float2(b.z, b.w), make_float2(acc.z, acc.w));
    acc = make_float4(lo.x, lo.y, hi.x, hi.y);
}
__device__ __forceinline__ void pfma(float4& acc, const float a, const float4 b) {
    const float2 aa = make_float2(a, a);
    const float2 lo = __ffma2_rn(aa, make_float2(b.x, b.y), make_float2(acc.x, acc.y));
    const float2 hi = __ffma2_rn(aa, make_float2(b.z, b.w), make_float2(acc.z, acc.w));
    acc = make_float4(lo.x, lo.y, hi.x, hi.y);
}
__device__ __forceinline__ float pmul(const float a, const float b) { return a * b; }
__device__ __forceinline__ void pfma(float& acc, const float a, const float b) { acc = fmaf(a, b, acc); }
// sum over the lane's channels of a * b
__device__ __forceinline__ float vdot(const float4 a, const float4 b) {
    return fmaf(a.w, b.w, fmaf(a.z, b.z, fmaf(a.y, b.y, a.x * b.x)));
}
__device__ __forceinline__ float vdot(const float2 a, const float2 b) { return fmaf(a.y, b.y, a.x * b.x); }
__device__ __forceinline__ float4 vadd(const float4 a, const float4 b) {
    return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
}
__device__ __forceinline__ float2 vadd(const float2 a, const float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ void vzero(float4& v) { v = make_float4(0.f, 0.f, 0.f, 0.f); }
__device__ __forceinline__ void vzero(float2& v) { v = make_float2(0.f, 0.f); }

// one channel per lane
__device__ __forceinline__ float vmul(const float a, const float b) { return a * b; }
__device__ __forceinline__ void vfma(float& acc, const float a, const float b) { acc = fmaf(a, b, acc); }
__device__ __forceinline__ float vdot(const float a, const float b) { return a * b; }
__device__ __forceinline__ float vadd(const float a, const float b) { return a + b; }
__device__ __forceinline__ void vzero(float& v) { v = 0.f; }
template <int V> struct VecOf;
template <> struct VecOf<1> { using type = float; };
template <> struct VecOf<4> { using type = float4; };
template <> struct VecOf<2> { using type = float2; };

// ---------------------------------------------------------------- mbarrier / bulk copy (PTX)
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// adds to the pending transaction count without arriving
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (and records the failure) if the phase does not complete within `limit` polls.
__device__ __forceinline__ bool mbar_wait_limit(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status,
                                                const uint32_t limit) {
#pragma unroll 1  // an unrolled spin loop only bloats the kernel text
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    if (status) atomicExch(status, kStatusTimeout);
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status) {
    return mbar_wait_limit(bar, parity, abort_flag, status, kSpinLimit);
}
// Contiguous global -> shared copy; both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_u32(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// ---------------------------------------------------------------- A-matrix tables
// For every (i0,i1) pair slot: where its records start and how many there are.
struct PairRec {
    int16_t start, count;
};

struct FwdParams {
    const float* x; const float* sh; const float* w;
    const float* vec;                  // edge vectors [E][3]: the kernel forms the harmonics itself (then sh is unused)
    const int32_t* senders; const int32_t* receivers;
    float* out;
    int64_t n_nodes, n_edges, chunk;   // chunk = edges per CTA (multiple of 4)
    float* partial;                    // [G][2][D*NQ] boundary-row partial sums
    int32_t* part_recv;                // [G][2] receiver of the head / tail partial, or -1
    int32_t* status;                   // device status word (0 = fine)
    int identity;                      // 1: every edge is its own sender and receiver (standalone tensor product)
    const int32_t* n_real;             // padded call: device word holding the number of real edges (else null)
    // fused double backward only: cotangents of grad_x, grad_sh, grad_w (laid out like x, sh, w)
    const float* ct_x; const float* ct_sh; const float* ct_w;
};

// Sums the pieces of every receiver row that was split between CTAs, in CTA order.
__global__ void fwd_fixup_kernel(int n_cta, int row_f4, const float4* __restrict__ partial,
                                 const int32_t* __restrict__ part_recv, float4* __restrict__ out);

// The edges this CTA works on.  Plain call: the host's split (n_edges, chunk).  Padded call: the number of real
// edges is only known on the device, so the equal split is formed here from *n_real.
__device__ __forceinline__ void cta_edge_range(const int64_t n_edges_host, const int64_t chunk_host,
                                               const int32_t* n_real, int64_t& n_edges, int64_t& chunk,
                                               int64_t& e_begin, int64_t& e_end) {
    n_edges = n_edges_host;
    chunk = chunk_host;
    if (n_real) {
        n_edges = min((int64_t)*n_real, n_edges_host);
        const int64_t per = (n_edges + gridDim.x - 1) / gridDim.x;
        chunk = max((int64_t)4, (per + 3) / 4 * 4);
    }
    e_begin = min(n_edges, (int64_t)blockIdx.x * chunk);
    e_end = min(n_edges, e_begin + chunk);
}

// Backward of a padded call: zero rows of grad_w and grad_sh for the padding edges [*n_real, n_edges).
__global__ void bwd_zero_padding_kernel(const int32_t* __restrict__ n_real, int64_t n_edges, int w_row_f4,
                                        int sh_row, float4* __restrict__ grad_w, float* __restrict__ grad_sh);

// Self-test of the bounded wait (e3j_selftest_bounded_wait): one warp waits on a barrier that nobody arrives on.
__global__ void bounded_wait_selftest_kernel(uint32_t limit, int32_t* status, int32_t* result);

// Backward pass 2: grad_x[a] = sum of the per-edge shares of the edges sent by a, in edge order.
__global__ void bwd_dx_reduce_kernel(int64_t n_nodes, int row_f4, const float4* __restrict__ dx_edge,
                                     const int32_t* __restrict__ sender_perm, const int32_t* __restrict__ colptr,
                                     float4* __restrict__ grad_x);

}  // namespace fast
}  // namespace e3j
