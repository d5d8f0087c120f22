// Slot tables of the convolution that forms its edge scalars in the kernel (fast_radial.cuh): the edges of
// every receiver padded to a multiple of 8 slots, so that a group of 8 slots never spans two receivers.
//   slotptr[b]     first slot of receiver b (exclusive scan of the padded degrees); slotptr[n_nodes] = slots
//   slot_edge[s]   edge id of slot s, or -1 for padding
//   group_recv[g]  receiver of group g = slots 8 g .. 8 g + 7
#include "fast_launch.cuh"
#include "fast_radial.cuh"

namespace e3j {
namespace fast {
namespace {

// One block: exclusive scan of pad8(rowptr[b + 1] - rowptr[b]) over the nodes.
__global__ void __launch_bounds__(1024) slot_scan_kernel(int64_t n_nodes, const int32_t* __restrict__ rowptr,
                                                         int32_t* __restrict__ slotptr) {
    __shared__ int sums[1024];
    const int tid = threadIdx.x;
    const int64_t per = (n_nodes + 1023) / 1024;
    const int64_t b0 = min(n_nodes, tid * per), b1 = min(n_nodes, b0 + per);
    int local = 0;
    for (int64_t b = b0; b < b1; ++b) local += (rowptr[b + 1] - rowptr[b] + kGroup - 1) / kGroup * kGroup;
    sums[tid] = local;
    __syncthreads();
    for (int off = 1; off < 1024; off <<= 1) {   // inclusive scan of the per-thread totals
        const int v = (tid >= off) ? sums[tid - off] : 0;
        __syncthreads();
        sums[tid] += v;
        __syncthreads();
    }
    int run = sums[tid] - local;
    for (int64_t b = b0; b < b1; ++b) {
        slotptr[b] = run;
        run += (rowptr[b + 1] - rowptr[b] + kGroup - 1) / kGroup * kGroup;
    }
    if (tid == 1023) slotptr[n_nodes] = sums[1023];
}

// One warp per receiver: its slots' edge ids and its groups' receiver id.
__global__ void slot_fill_kernel(int64_t n_nodes, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ slotptr,
                                 int32_t* __restrict__ slot_edge, int32_t* __restrict__ group_recv) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t b = warp; b < n_nodes; b += n_warps) {
        const int e0 = rowptr[b], deg = rowptr[b + 1] - e0;
        const int s0 = slotptr[b], n_slots = slotptr[b + 1] - s0;
        for (int i = lane; i < n_slots; i += 32) {
            slot_edge[s0 + i] = (i < deg) ? e0 + i : -1;
            if (i % kGroup == 0) group_recv[(s0 + i) / kGroup] = (int32_t)b;
        }
    }
}

}  // namespace

int build_slot_tables(int64_t n_nodes, int64_t n_edges, const int32_t* rowptr, int32_t* slotptr, int32_t* slot_edge,
                      int32_t* group_recv, cudaStream_t st) {
    (void)n_edges;
    slot_scan_kernel<<<1, 1024, 0, st>>>(n_nodes, rowptr, slotptr);
    if (int s = after_launch()) return s;
    const int blocks = (int)std::min<int64_t>((n_nodes + 7) / 8, 8 * (int64_t)sm_count());
    slot_fill_kernel<<<std::max(blocks, 1), 256, 0, st>>>(n_nodes, rowptr, slotptr, slot_edge, group_recv);
    return after_launch();
}

}  // namespace fast
}  // namespace e3j

