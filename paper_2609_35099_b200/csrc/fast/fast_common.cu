// Kernels shared by all signature-specialised entries.
#include "fast_common.cuh"

namespace e3j {
namespace fast {

__global__ void fwd_fixup_kernel(int n_cta, int row_f4, const float4* __restrict__ partial,
                                 const int32_t* __restrict__ part_recv, float4* __restrict__ out) {
    grid_dependency_wait();
    const int c = blockIdx.x;
    const int b = part_recv[2 * c + 1];  // a row whose first piece is this CTA's tail
    if (b < 0) return;
    int last = c;
    while (last + 1 < n_cta && part_recv[2 * (last + 1)] == b) ++last;
    for (int i = threadIdx.x; i < row_f4; i += blockDim.x) {
        float4 sum = partial[(size_t)(2 * c + 1) * row_f4 + i];
        for (int c2 = c + 1; c2 <= last; ++c2) {
            const float4 v = partial[(size_t)(2 * c2) * row_f4 + i];
            sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
        }
        out[(size_t)b * row_f4 + i] = sum;
    }
}

// One warp, one barrier with one expected arrival that never comes, no copy in flight: the wait runs out after
// `limit` polls, records the time-out in *status and returns false; result[0] = what the wait returned,
// result[1] = the CTA's abort flag afterwards.  Nothing here can hang: the loop is bounded by `limit`.
__global__ void bounded_wait_selftest_kernel(uint32_t limit, int32_t* status, int32_t* result) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) { mbar_init(&bar, 1); abort_flag = 0; mbar_fence_init(); }
    __syncthreads();
    const bool ok = mbar_wait_limit(&bar, 0, &abort_flag, status, limit);
    __syncthreads();
    if (threadIdx.x == 0) { result[0] = ok ? 1 : 0; result[1] = abort_flag; }
}

__global__ void bwd_zero_padding_kernel(const int32_t* __restrict__ n_real, int64_t n_edges, int w_row_f4,
                                        int sh_row, float4* __restrict__ grad_w, float* __restrict__ grad_sh) {
    const int64_t first = min((int64_t)*n_real, n_edges);
    const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int64_t e = first + blockIdx.x; e < n_edges; e += gridDim.x) {
        if (grad_w)
            for (int i = threadIdx.x; i < w_row_f4; i += blockDim.x) grad_w[(size_t)e * w_row_f4 + i] = z;
        if (grad_sh)
            for (int i = threadIdx.x; i < sh_row; i += blockDim.x) grad_sh[(size_t)e * sh_row + i] = 0.f;
    }
}

__global__ void bwd_dx_reduce_kernel(int64_t n_nodes, int row_f4, const float4* __restrict__ dx_edge,
                                     const int32_t* __restrict__ sender_perm, const int32_t* __restrict__ colptr,
                                     float4* __restrict__ grad_x) {
    grid_dependency_wait();
    for (int64_t a = blockIdx.x; a < n_nodes; a += gridDim.x) {
        const int j0 = colptr[a], j1 = colptr[a + 1];
        for (int i = threadIdx.x; i < row_f4; i += blockDim.x) {
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            int j = j0;
            // eight independent loads in flight; the additions stay in edge order
            for (; j + 8 <= j1; j += 8) {
                float4 v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = dx_edge[(size_t)sender_perm[j + u] * row_f4 + i];
#pragma unroll
                for (int u = 0; u < 8; ++u) { acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w; }
            }
            for (; j < j1; ++j) {
                const float4 v = dx_edge[(size_t)sender_perm[j] * row_f4 + i];
                acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
            }
            grad_x[(size_t)a * row_f4 + i] = acc;
        }
    }
}

__global__ void bwd_rows_reduce_kernel(int64_t n_nodes, int row_f4, const float4* __restrict__ dx_rows,
                                       const int32_t* __restrict__ row_ptr, float4* __restrict__ grad_x) {
    grid_dependency_wait();
    for (int64_t a = blockIdx.x; a < n_nodes; a += gridDim.x) {
        const int j0 = row_ptr[a], j1 = row_ptr[a + 1];
        for (int i = threadIdx.x; i < row_f4; i += blockDim.x) {
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            int j = j0;
            for (; j + 8 <= j1; j += 8) {   // eight independent loads in flight; the additions stay in row order
                float4 v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = dx_rows[(size_t)(j + u) * row_f4 + i];
#pragma unroll
                for (int u = 0; u < 8; ++u) { acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w; }
            }
            for (; j < j1; ++j) {
                const float4 v = dx_rows[(size_t)j * row_f4 + i];
                acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
            }
            grad_x[(size_t)a * row_f4 + i] = acc;
        }
    }
}

}  // namespace fast
}  // namespace e3j

