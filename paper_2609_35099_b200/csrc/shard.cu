// Receiver sharding across GPUs (one process per GPU): the integer kernels that turn a rank's slice of the edge
// list into a local problem, and the two row kernels of its halo exchange.
//
// A rank owns the receivers [node_lo, node_hi) and every edge into them (a contiguous slice of the
// receiver-sorted edge list).  Local node ids: owned nodes first, node_lo + i -> i; then the halo, the senders
// of the slice that the rank does not own, in ascending global id: halo_ids[h] -> (node_hi - node_lo) + h.
#include "common.cuh"

namespace e3j {
namespace {

__global__ void shard_mark_kernel(int64_t n_edges, int32_t lo, int32_t hi, const int32_t* __restrict__ senders,
                                  int32_t* __restrict__ flag) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < n_edges; e += stride) {
        const int32_t s = senders[e];
        if (s < lo || s >= hi) flag[s] = 1;   // every writer stores the same value
    }
}

// One block: exclusive scan of flag[0 .. n) into pos, halo_ids[pos[s]] = s where flagged, *n_halo = total.
__global__ void __launch_bounds__(1024) shard_scan_kernel(int64_t n, const int32_t* __restrict__ flag,
                                                          int32_t* __restrict__ pos, int32_t* __restrict__ halo_ids,
                                                          int32_t* __restrict__ n_halo) {
    __shared__ int sums[1024];
    const int tid = threadIdx.x;
    const int64_t per = (n + 1023) / 1024;
    const int64_t b0 = min(n, tid * per), b1 = min(n, b0 + per);
    int local = 0;
    for (int64_t b = b0; b < b1; ++b) local += flag[b];
    sums[tid] = local;
    __syncthreads();
    for (int off = 1; off < 1024; off <<= 1) {
        const int v = (tid >= off) ? sums[tid - off] : 0;
        __syncthreads();
        sums[tid] += v;
        __syncthreads();
    }
    int run = sums[tid] - local;
    for (int64_t b = b0; b < b1; ++b) {
        pos[b] = run;
        if (flag[b]) halo_ids[run++] = (int32_t)b;
    }
    if (tid == 1023) *n_halo = sums[1023];
}

__global__ void shard_renumber_kernel(int64_t n_edges, int32_t lo, int32_t hi, const int32_t* __restrict__ senders,
                                      const int32_t* __restrict__ receivers, const int32_t* __restrict__ pos,
                                      int32_t* __restrict__ local_senders, int32_t* __restrict__ local_receivers) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < n_edges; e += stride) {
        const int32_t s = senders[e];
        local_senders[e] = (s >= lo && s < hi) ? s - lo : (hi - lo) + pos[s];
        local_receivers[e] = receivers[e] - lo;
    }
}

// dst[i, :] = src[ids[i], :]   /   dst[ids[i], :] += src[i, :]  (ids unique within a call: no two rows collide)
template <bool ADD>
__global__ void rows_kernel(float4* __restrict__ dst, const float4* __restrict__ src, const int32_t* __restrict__ ids,
                            int64_t n_ids, int row_f4) {
    for (int64_t i = blockIdx.x; i < n_ids; i += gridDim.x) {
        const int64_t r = ids[i];
        for (int c = threadIdx.x; c < row_f4; c += blockDim.x) {
            if (ADD) {
                float4 a = dst[r * row_f4 + c];
                const float4 b = src[i * row_f4 + c];
                a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
                dst[r * row_f4 + c] = a;
            } else {
                dst[i * row_f4 + c] = src[r * row_f4 + c];
            }
        }
    }
}

inline int blocks(int64_t n, int threads) {
    return (int)std::max<int64_t>(1, std::min<int64_t>((n + threads - 1) / threads, (int64_t)sm_count() * 16));
}

}  // namespace
}  // namespace e3j

using namespace e3j;

extern "C" {

size_t e3j_shard_prepare_workspace_bytes(int64_t n_nodes) {
    return n_nodes < 0 ? 0 : 2 * align_up(4 * (size_t)(n_nodes + 1), 256);   // flag, pos
}

int e3j_shard_prepare(int64_t n_nodes, int64_t n_edges_shard, int32_t node_lo, int32_t node_hi,
                      const int32_t* senders, const int32_t* receivers, int32_t* local_senders,
                      int32_t* local_receivers, int32_t* halo_ids, int32_t* n_halo, void* workspace,
                      size_t workspace_bytes, void* stream) {
    if (n_nodes < 0 || n_edges_shard < 0 || node_lo < 0 || node_hi < node_lo || node_hi > n_nodes ||
        n_nodes >= (1ll << 31) - 1 || n_edges_shard >= (1ll << 31) - 1)
        return E3J_ERR_INVALID_ARG;
    if (!halo_ids || !n_halo) return E3J_ERR_INVALID_ARG;
    if (n_edges_shard > 0 && (!senders || !receivers || !local_senders || !local_receivers)) return E3J_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255u) || workspace_bytes < e3j_shard_prepare_workspace_bytes(n_nodes))
        return E3J_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    int32_t* flag = (int32_t*)workspace;
    int32_t* pos = (int32_t*)((char*)workspace + align_up(4 * (size_t)(n_nodes + 1), 256));
    E3J_CUDA_TRY(cudaMemsetAsync(flag, 0, 4 * (size_t)(n_nodes + 1), st));
    if (n_edges_shard > 0) {
        shard_mark_kernel<<<blocks(n_edges_shard, 256), 256, 0, st>>>(n_edges_shard, node_lo, node_hi, senders, flag);
        if (int s = after_launch()) return s;
    }
    shard_scan_kernel<<<1, 1024, 0, st>>>(n_nodes, flag, pos, halo_ids, n_halo);
    if (int s = after_launch()) return s;
    if (n_edges_shard > 0) {
        shard_renumber_kernel<<<blocks(n_edges_shard, 256), 256, 0, st>>>(n_edges_shard, node_lo, node_hi, senders,
                                                                         receivers, pos, local_senders, local_receivers);
        if (int s = after_launch()) return s;
    }
    return E3J_OK;
}

static int rows_call(bool add, float* dst, const float* src, const int32_t* ids, int64_t n_ids, int64_t row_len,
                     void* stream) {
    if (n_ids < 0 || row_len <= 0 || row_len % 4 != 0) return E3J_ERR_INVALID_ARG;
    if (n_ids == 0) return E3J_OK;
    if (!dst || !src || !ids || (((uintptr_t)dst | (uintptr_t)src) & 15u)) return E3J_ERR_INVALID_ARG;
    const int row_f4 = (int)(row_len / 4);
    const int threads = std::min(256, std::max(32, (row_f4 + 31) / 32 * 32));
    const int grid = (int)std::min<int64_t>(n_ids, (int64_t)sm_count() * 32);
    if (add)
        rows_kernel<true><<<grid, threads, 0, (cudaStream_t)stream>>>((float4*)dst, (const float4*)src, ids, n_ids, row_f4);
    else
        rows_kernel<false><<<grid, threads, 0, (cudaStream_t)stream>>>((float4*)dst, (const float4*)src, ids, n_ids, row_f4);
    return after_launch();
}

int e3j_rows_gather(float* dst, const float* src, const int32_t* ids, int64_t n_ids, int64_t row_len, void* stream) {
    return rows_call(false, dst, src, ids, n_ids, row_len, stream);
}

int e3j_rows_add(float* dst, const float* src, const int32_t* ids, int64_t n_ids, int64_t row_len, void* stream) {
    return rows_call(true, dst, src, ids, n_ids, row_len, stream);
}

}  // extern "C"
