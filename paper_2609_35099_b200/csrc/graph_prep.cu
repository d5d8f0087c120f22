// Graph preparation on the device: receiver CSR pointers and the sender-sorted edge
// permutation used by the backward ("message passing on the transposed graph").
// Integer work only; integer atomics are used to claim slots, and every bucket is
// sorted afterwards so the result does not depend on the order they were claimed in.
#include "common.cuh"

namespace e3j {
namespace {

__global__ void rowptr_kernel(int64_t n_nodes, int64_t n_edges, const int32_t* __restrict__ receivers,
                              int32_t* __restrict__ rowptr) {
    for (int64_t b = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; b <= n_nodes;
         b += (int64_t)gridDim.x * blockDim.x) {
        int64_t lo = 0, hi = n_edges;  // first edge with receiver >= b
        while (lo < hi) {
            const int64_t mid = (lo + hi) >> 1;
            if (receivers[mid] < b) lo = mid + 1; else hi = mid;
        }
        rowptr[b] = (int32_t)lo;
    }
}

// `pad_recv`: when not null, edges whose receiver id is >= n_nodes are padding and are left out.
__global__ void count_senders_kernel(int64_t n_nodes, int64_t n_edges, const int32_t* __restrict__ senders,
                                     const int32_t* __restrict__ pad_recv, int32_t* __restrict__ colptr) {
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < n_edges;
         e += (int64_t)gridDim.x * blockDim.x) {
        if (pad_recv && pad_recv[e] >= n_nodes) continue;
        atomicAdd(&colptr[senders[e]], 1);
    }
}

// In-place exclusive scan of v[0..n) by one block; v[n] receives the total.
__global__ void __launch_bounds__(1024) exclusive_scan_kernel(int64_t n, int32_t* __restrict__ v) {
    __shared__ int32_t warp_sums[32];
    __shared__ int32_t carry_s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    for (int64_t base = 0; base < n; base += blockDim.x) {
        const int64_t i = base + threadIdx.x;
        const int32_t mine = (i < n) ? v[i] : 0;
        int32_t incl = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int32_t up = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += up;
        }
        if (lane == 31) warp_sums[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int32_t ws = warp_sums[lane];
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int32_t up = __shfl_up_sync(0xffffffffu, ws, off);
                if (lane >= off) ws += up;
            }
            warp_sums[lane] = ws;  // inclusive over warps
        }
        __syncthreads();
        const int32_t carry = carry_s;
        const int32_t before = carry + (warp ? warp_sums[warp - 1] : 0) + incl - mine;
        if (i < n) v[i] = before;
        __syncthreads();
        if (threadIdx.x == blockDim.x - 1) carry_s = before + mine;
        __syncthreads();
    }
    if (threadIdx.x == 0) v[n] = carry_s;
}

// Claims a slot for every edge; afterwards colptr[a] is the END of bucket a.
__global__ void fill_kernel(int64_t n_nodes, int64_t n_edges, const int32_t* __restrict__ senders,
                            const int32_t* __restrict__ pad_recv, int32_t* __restrict__ colptr,
                            int32_t* __restrict__ perm) {
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < n_edges;
         e += (int64_t)gridDim.x * blockDim.x) {
        if (pad_recv && pad_recv[e] >= n_nodes) continue;
        const int32_t pos = atomicAdd(&colptr[senders[e]], 1);
        perm[pos] = (int32_t)e;
    }
}

__device__ inline void sift_down(int32_t* v, int64_t root, int64_t n) {
    while (true) {
        int64_t child = 2 * root + 1;
        if (child >= n) return;
        if (child + 1 < n && v[child + 1] > v[child]) ++child;
        if (v[root] >= v[child]) return;
        const int32_t tmp = v[root]; v[root] = v[child]; v[child] = tmp;
        root = child;
    }
}

// Sorts every bucket ascending by edge id.  colptr holds bucket ENDS here.
// One warp per bucket.  Edge ids are distinct, so an element's place is the number of smaller ones: buckets
// of up to kRankMax entries are staged in shared memory and every lane counts the ranks of its elements;
// a longer bucket (a hub sender) is heap-sorted in place by one lane.
constexpr int kRankMax = 1024;
constexpr int kSortWarps = 4;

__global__ void __launch_bounds__(32 * kSortWarps)
sort_buckets_kernel(int64_t n_nodes, const int32_t* __restrict__ colptr, int32_t* __restrict__ perm) {
    __shared__ int32_t stage[kSortWarps][kRankMax];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int32_t* mine = stage[warp];
    for (int64_t a = (int64_t)blockIdx.x * kSortWarps + warp; a < n_nodes; a += (int64_t)gridDim.x * kSortWarps) {
        const int64_t begin = a ? colptr[a - 1] : 0, n = colptr[a] - begin;
        int32_t* v = perm + begin;
        if (n <= 1) continue;
        if (n <= kRankMax) {
            for (int i = lane; i < n; i += 32) mine[i] = v[i];
            __syncwarp();
            for (int i = lane; i < n; i += 32) {
                const int32_t key = mine[i];
                int rank = 0;
                for (int j = 0; j < n; ++j) rank += mine[j] < key;
                v[rank] = key;
            }
            __syncwarp();
        } else if (lane == 0) {
            for (int64_t i = n / 2 - 1; i >= 0; --i) sift_down(v, i, n);
            for (int64_t end = n - 1; end > 0; --end) {
                const int32_t tmp = v[0]; v[0] = v[end]; v[end] = tmp;
                sift_down(v, 0, end);
            }
        }
    }
}

// colptr[a] (end of bucket a) -> colptr[a+1]; colptr[0] = 0.  One block, top down.
__global__ void __launch_bounds__(1024) shift_up_kernel(int64_t n_nodes, int32_t* __restrict__ colptr) {
    for (int64_t hi = n_nodes; hi > 0; hi -= blockDim.x) {
        const int64_t i = hi - 1 - threadIdx.x;  // source index
        int32_t val = 0;
        if (i >= 0) val = colptr[i];
        __syncthreads();
        if (i >= 0) colptr[i + 1] = val;
        __syncthreads();
    }
    if (threadIdx.x == 0) colptr[0] = 0;
}

__global__ void validate_kernel(int64_t n_nodes, int64_t n_edges, const int32_t* __restrict__ senders,
                                const int32_t* __restrict__ receivers, int32_t* __restrict__ status) {
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < n_edges;
         e += (int64_t)gridDim.x * blockDim.x) {
        const int32_t s = senders[e], r = receivers[e];
        bool bad = s < 0 || s >= n_nodes || r < 0 || r >= n_nodes;
        if (e > 0 && receivers[e - 1] > r) bad = true;
        if (bad) *status = E3J_ERR_GRAPH;  // every writer stores the same value
    }
}

inline int blocks_for(int64_t n, int threads) {
    int64_t b = (n + threads - 1) / threads;
    if (b < 1) b = 1;
    if (b > sm_count() * 16) b = sm_count() * 16;
    return (int)b;
}

}  // namespace

int graph_prepare(int64_t n_nodes, int64_t n_edges, const int32_t* senders, const int32_t* receivers,
                  int32_t* rowptr, int32_t* sender_perm, int32_t* colptr, cudaStream_t st, bool padded) {
    const int32_t* pad_recv = padded ? receivers : nullptr;
    if (rowptr) {
        rowptr_kernel<<<blocks_for(n_nodes + 1, 256), 256, 0, st>>>(n_nodes, n_edges, receivers, rowptr);
        if (int s = after_launch()) return s;
    }
    if (sender_perm && colptr) {
        E3J_CUDA_TRY(cudaMemsetAsync(colptr, 0, sizeof(int32_t) * (size_t)(n_nodes + 1), st));
        if (n_edges > 0) {
            count_senders_kernel<<<blocks_for(n_edges, 256), 256, 0, st>>>(n_nodes, n_edges, senders, pad_recv, colptr);
            if (int s = after_launch()) return s;
        }
        exclusive_scan_kernel<<<1, 1024, 0, st>>>(n_nodes, colptr);
        if (int s = after_launch()) return s;
        if (n_edges > 0) {
            fill_kernel<<<blocks_for(n_edges, 256), 256, 0, st>>>(n_nodes, n_edges, senders, pad_recv, colptr,
                                                               sender_perm);
            if (int s = after_launch()) return s;
            sort_buckets_kernel<<<blocks_for(n_nodes, kSortWarps), 32 * kSortWarps, 0, st>>>(n_nodes, colptr, sender_perm);
            if (int s = after_launch()) return s;
            shift_up_kernel<<<1, 1024, 0, st>>>(n_nodes, colptr);
            if (int s = after_launch()) return s;
        }
    }
    return E3J_OK;
}

int graph_validate(int64_t n_nodes, int64_t n_edges, const int32_t* senders, const int32_t* receivers,
                   int32_t* status, cudaStream_t st) {
    E3J_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), st));
    if (n_edges > 0) {
        validate_kernel<<<blocks_for(n_edges, 256), 256, 0, st>>>(n_nodes, n_edges, senders, receivers, status);
        if (int s = after_launch()) return s;
    }
    return E3J_OK;
}

}  // namespace e3j
