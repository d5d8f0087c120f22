// Table-driven kernels that work for every plan (any irreps, any channel count).
//
// Each output element is owned by exactly one thread and is computed as the
// defining sum in a fixed order, so the results are deterministic without
// atomics.  This is the paper's "transposed record sets" formulation (section
// "Differentiation": for dx the records are sorted by i1, for dy by i2): every
// cotangent is a gather with its own sorted copy of the coefficient records.
// They are the fallback for signatures that have no specialised kernel and the
// on-device cross-check for the specialised ones.
#pragma once
#include "common.cuh"

namespace e3j {
namespace generic {

// IDENT = true: every row is its own sender and receiver (standalone tensor product).

template <bool IDENT>
__global__ void __launch_bounds__(256)
conv_fwd_kernel(DeviceTables t, Dims dm, int64_t n_nodes, const float* __restrict__ x,
                const float* __restrict__ sh, const float* __restrict__ w,
                const int32_t* __restrict__ senders, const int32_t* __restrict__ rowptr,
                float* __restrict__ out) {
    const int per_node = dm.D * dm.nq;
    for (int64_t b = blockIdx.x; b < n_nodes; b += gridDim.x) {
        const int64_t e0 = IDENT ? b : rowptr[b];
        const int64_t e1 = IDENT ? b + 1 : rowptr[b + 1];
        for (int idx = threadIdx.x; idx < per_node; idx += blockDim.x) {
            const int i0 = idx / dm.nq, q = idx - i0 * dm.nq;
            const int k = t.i0_path[i0];
            const int r0 = t.i0_start[i0], r1 = t.i0_start[i0 + 1];
            float acc = 0.f;
            for (int64_t e = e0; e < e1; ++e) {
                const int64_t a = IDENT ? e : (int64_t)senders[e];
                const float* xa = x + (size_t)a * dm.d * dm.nq + q;
                const float* ye = sh + (size_t)e * dm.dp;
                float z = 0.f;
                for (int r = r0; r < r1; ++r) {
                    const PackedRecord rc = t.by_i0[r];
                    z = fmaf(rc.val * ye[rc.b], xa[(size_t)rc.a * dm.nq], z);
                }
                acc = fmaf(w[((size_t)e * dm.P + k) * dm.nq + q], z, acc);
            }
            out[((size_t)b * dm.D + i0) * dm.nq + q] = acc;
        }
    }
}

// Edge-local cotangents: grad_w[e,k,q] and grad_sh[e,i2]; one block per edge.
template <bool IDENT>
__global__ void __launch_bounds__(256)
conv_bwd_edge_kernel(DeviceTables t, Dims dm, int64_t n_edges, const float* __restrict__ x,
                     const float* __restrict__ sh, const float* __restrict__ w,
                     const int32_t* __restrict__ senders, const int32_t* __restrict__ receivers,
                     const float* __restrict__ g, float* __restrict__ grad_w,
                     float* __restrict__ grad_sh, const int32_t* __restrict__ n_real) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    // padded call: edges from *n_real on are padding; their gradient rows are zero and nothing of them is read
    const int64_t n_live = n_real ? min((int64_t)*n_real, n_edges) : n_edges;
    for (int64_t e = blockIdx.x; e < n_edges; e += gridDim.x) {
        if (e >= n_live) {
            if (grad_w)
                for (int idx = threadIdx.x; idx < dm.P * dm.nq; idx += blockDim.x)
                    grad_w[(size_t)e * dm.P * dm.nq + idx] = 0.f;
            if (grad_sh && threadIdx.x < dm.dp) grad_sh[(size_t)e * dm.dp + threadIdx.x] = 0.f;
            continue;
        }
        const int64_t a = IDENT ? e : (int64_t)senders[e];
        const int64_t b = IDENT ? e : (int64_t)receivers[e];
        const float* xa = x + (size_t)a * dm.d * dm.nq;
        const float* gb = g + (size_t)b * dm.D * dm.nq;
        const float* ye = sh + (size_t)e * dm.dp;
        const float* we = w + (size_t)e * dm.P * dm.nq;
        if (grad_w) {
            for (int idx = threadIdx.x; idx < dm.P * dm.nq; idx += blockDim.x) {
                const int k = idx / dm.nq, q = idx - k * dm.nq;
                float sum = 0.f;
                for (int i0 = t.path_out_off[k]; i0 < t.path_out_off[k + 1]; ++i0) {
                    float z = 0.f;
                    for (int r = t.i0_start[i0]; r < t.i0_start[i0 + 1]; ++r) {
                        const PackedRecord rc = t.by_i0[r];
                        z = fmaf(rc.val * ye[rc.b], xa[(size_t)rc.a * dm.nq + q], z);
                    }
                    sum = fmaf(gb[(size_t)i0 * dm.nq + q], z, sum);
                }
                grad_w[((size_t)e * dm.P + k) * dm.nq + q] = sum;
            }
        }
        if (grad_sh) {
            for (int i2 = warp; i2 < dm.dp; i2 += nwarps) {
                float part = 0.f;
                for (int q = lane; q < dm.nq; q += 32) {
                    float s = 0.f;
                    for (int r = t.i2_start[i2]; r < t.i2_start[i2 + 1]; ++r) {
                        const PackedRecord rc = t.by_i2[r];  // (i0, i1, path)
                        s = fmaf(rc.val * xa[(size_t)rc.b * dm.nq + q],
                                 we[(size_t)rc.c * dm.nq + q] * gb[(size_t)rc.a * dm.nq + q], s);
                    }
                    part += s;
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
                if (lane == 0) grad_sh[(size_t)e * dm.dp + i2] = part;
            }
        }
    }
}

// Sender cotangent: grad_x[a,i1,q] gathers over the edges sent by a, in edge order.
template <bool IDENT>
__global__ void __launch_bounds__(256)
conv_bwd_node_kernel(DeviceTables t, Dims dm, int64_t n_nodes, const float* __restrict__ sh,
                     const float* __restrict__ w, const int32_t* __restrict__ receivers,
                     const int32_t* __restrict__ sender_perm, const int32_t* __restrict__ colptr,
                     const float* __restrict__ g, float* __restrict__ grad_x) {
    const int per_node = dm.d * dm.nq;
    for (int64_t a = blockIdx.x; a < n_nodes; a += gridDim.x) {
        const int64_t j0 = IDENT ? a : colptr[a];
        const int64_t j1 = IDENT ? a + 1 : colptr[a + 1];
        for (int idx = threadIdx.x; idx < per_node; idx += blockDim.x) {
            const int i1 = idx / dm.nq, q = idx - i1 * dm.nq;
            const int r0 = t.i1_start[i1], r1 = t.i1_start[i1 + 1];
            float acc = 0.f;
            for (int64_t j = j0; j < j1; ++j) {
                const int64_t e = IDENT ? j : (int64_t)sender_perm[j];
                const int64_t b = IDENT ? e : (int64_t)receivers[e];
                const float* gb = g + (size_t)b * dm.D * dm.nq + q;
                const float* ye = sh + (size_t)e * dm.dp;
                const float* we = w + (size_t)e * dm.P * dm.nq + q;
                float s = 0.f;
                for (int r = r0; r < r1; ++r) {
                    const PackedRecord rc = t.by_i1[r];  // (i0, i2, path)
                    s = fmaf(rc.val * ye[rc.b], we[(size_t)rc.c * dm.nq] * gb[(size_t)rc.a * dm.nq], s);
                }
                acc += s;
            }
            grad_x[((size_t)a * dm.d + i1) * dm.nq + q] = acc;
        }
    }
}

}  // namespace generic
}  // namespace e3j
