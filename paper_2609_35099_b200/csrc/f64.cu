// Float64 entry points (the paper ships float64 builds of its kernels beside the float32 ones).
//
// Table-driven kernels in double precision, for any plan: every output element is owned by one thread and is the
// defining sum in a fixed order (edges in list order, records in table order), with the coefficient values kept
// in float64 as the plan builder computed them.  They are the float64 counterpart of generic_kernels.cuh, one
// channel per thread; there are no signature-specialised float64 kernels.
#include "common.cuh"

namespace e3j {

int graph_prepare(int64_t, int64_t, const int32_t*, const int32_t*, int32_t*, int32_t*, int32_t*, cudaStream_t,
                  bool padded = false);

namespace {

__global__ void __launch_bounds__(256)
fwd_f64_kernel(DeviceTables t, Dims dm, int64_t n_nodes, const double* __restrict__ x, const double* __restrict__ sh,
               const double* __restrict__ w, const int32_t* __restrict__ senders, const int32_t* __restrict__ rowptr,
               double* __restrict__ out) {
    const int per_node = dm.D * dm.nq;
    for (int64_t b = blockIdx.x; b < n_nodes; b += gridDim.x) {
        const int64_t e0 = rowptr[b], e1 = rowptr[b + 1];
        for (int idx = threadIdx.x; idx < per_node; idx += blockDim.x) {
            const int i0 = idx / dm.nq, q = idx - i0 * dm.nq;
            const int r0 = t.i0_start[i0], r1 = t.i0_start[i0 + 1];
            double acc = 0.0;
            for (int64_t e = e0; e < e1; ++e) {
                const double* xa = x + (size_t)senders[e] * dm.d * dm.nq + q;
                const double* ye = sh + (size_t)e * dm.dp;
                const double* we = w + (size_t)e * dm.P * dm.nq + q;
                double z = 0.0;
                for (int r = r0; r < r1; ++r) {
                    const PackedRecord rc = t.by_i0[r];   // (i1, i2, path)
                    z = fma(t.val64_i0[r] * ye[rc.b], we[(size_t)rc.c * dm.nq] * xa[(size_t)rc.a * dm.nq], z);
                }
                acc += z;
            }
            out[((size_t)b * dm.D + i0) * dm.nq + q] = acc;
        }
    }
}

// grad_w[e,k,q] and grad_sh[e,i2]; one block per edge
__global__ void __launch_bounds__(256)
bwd_edge_f64_kernel(DeviceTables t, Dims dm, int64_t n_edges, const double* __restrict__ x, const double* __restrict__ sh,
                    const double* __restrict__ w, const int32_t* __restrict__ senders,
                    const int32_t* __restrict__ receivers, const double* __restrict__ g, double* __restrict__ grad_w,
                    double* __restrict__ grad_sh) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int64_t e = blockIdx.x; e < n_edges; e += gridDim.x) {
        const double* xa = x + (size_t)senders[e] * dm.d * dm.nq;
        const double* gb = g + (size_t)receivers[e] * dm.D * dm.nq;
        const double* ye = sh + (size_t)e * dm.dp;
        const double* we = w + (size_t)e * dm.P * dm.nq;
        if (grad_w) {
            for (int idx = threadIdx.x; idx < dm.P * dm.nq; idx += blockDim.x) {
                const int k = idx / dm.nq, q = idx - k * dm.nq;
                double sum = 0.0;
                const int row0 = t.path_out_off[k];
                for (int i0 = row0; i0 < row0 + t.path_rows[k]; ++i0) {
                    double z = 0.0;
                    for (int r = t.i0_start[i0]; r < t.i0_start[i0 + 1]; ++r) {
                        const PackedRecord rc = t.by_i0[r];
                        if (rc.c != k) continue;   // (a collapsed plan has other paths' records on this row)
                        z = fma(t.val64_i0[r] * ye[rc.b], xa[(size_t)rc.a * dm.nq + q], z);
                    }
                    sum = fma(gb[(size_t)i0 * dm.nq + q], z, sum);
                }
                grad_w[(size_t)e * dm.P * dm.nq + idx] = sum;
            }
        }
        if (grad_sh) {
            for (int i2 = warp; i2 < dm.dp; i2 += nwarps) {
                double part = 0.0;
                for (int q = lane; q < dm.nq; q += 32) {
                    double s = 0.0;
                    for (int r = t.i2_start[i2]; r < t.i2_start[i2 + 1]; ++r) {
                        const PackedRecord rc = t.by_i2[r];   // (i0, i1, path)
                        s = fma(t.val64_i2[r] * xa[(size_t)rc.b * dm.nq + q],
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

// grad_x[a,i1,q] gathers over the edges sent by a, in edge order
__global__ void __launch_bounds__(256)
bwd_node_f64_kernel(DeviceTables t, Dims dm, int64_t n_nodes, const double* __restrict__ sh, const double* __restrict__ w,
                    const int32_t* __restrict__ receivers, const int32_t* __restrict__ sender_perm,
                    const int32_t* __restrict__ colptr, const double* __restrict__ g, double* __restrict__ grad_x) {
    const int per_node = dm.d * dm.nq;
    for (int64_t a = blockIdx.x; a < n_nodes; a += gridDim.x) {
        for (int idx = threadIdx.x; idx < per_node; idx += blockDim.x) {
            const int i1 = idx / dm.nq, q = idx - i1 * dm.nq;
            double acc = 0.0;
            for (int64_t j = colptr[a]; j < colptr[a + 1]; ++j) {
                const int64_t e = sender_perm[j];
                const double* gb = g + (size_t)receivers[e] * dm.D * dm.nq + q;
                const double* ye = sh + (size_t)e * dm.dp;
                const double* we = w + (size_t)e * dm.P * dm.nq + q;
                double s = 0.0;
                for (int r = t.i1_start[i1]; r < t.i1_start[i1 + 1]; ++r) {
                    const PackedRecord rc = t.by_i1[r];   // (i0, i2, path)
                    s = fma(t.val64_i1[r] * ye[rc.b], we[(size_t)rc.c * dm.nq] * gb[(size_t)rc.a * dm.nq], s);
                }
                acc += s;
            }
            grad_x[((size_t)a * dm.d + i1) * dm.nq + q] = acc;
        }
    }
}

inline int grid_for(int64_t n) { return (int)std::min<int64_t>(std::max<int64_t>(n, 1), (int64_t)sm_count() * 32); }

bool basic_args_ok(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges) {
    return plan && n_nodes >= 0 && n_edges >= 0 && n_nodes < (1ll << 31) - 1 && n_edges < (1ll << 31) - 1;
}

}  // namespace
}  // namespace e3j

using namespace e3j;

extern "C" {

size_t e3j_conv_f64_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges) {
    if (!plan || n_nodes < 0 || n_edges < 0) return 0;
    return 2 * align_up(4 * (size_t)(n_nodes + 1), 256) + align_up(4 * (size_t)std::max<int64_t>(n_edges, 1), 256);
}

int e3j_conv_fwd_f64(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const double* x, const double* sh,
                     const double* w, const int32_t* senders, const int32_t* receivers, const int32_t* rowptr,
                     double* out, void* workspace, size_t workspace_bytes, void* stream) {
    if (!basic_args_ok(plan, n_nodes, n_edges)) return E3J_ERR_INVALID_ARG;
    if (n_nodes == 0) return E3J_OK;
    if (!x || !out || (n_edges > 0 && (!sh || !w || !senders || !receivers))) return E3J_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (!rowptr) {
        if (!workspace || ((uintptr_t)workspace & 255u) || workspace_bytes < e3j_conv_f64_workspace_bytes(plan, n_nodes, n_edges))
            return E3J_ERR_WORKSPACE;
        int32_t* rp = (int32_t*)workspace;
        if (int s = graph_prepare(n_nodes, n_edges, senders, receivers, rp, nullptr, nullptr, st)) return s;
        rowptr = rp;
    }
    DeviceTables t;
    if (int s = get_device_tables(plan, t)) return s;
    const Dims dm{plan->nq, plan->d, plan->dp, plan->P, plan->D, (plan->flags & E3J_PLAN_COLLAPSE_OUTPUTS) ? 1 : 0};
    fwd_f64_kernel<<<grid_for(n_nodes), 256, 0, st>>>(t, dm, n_nodes, x, sh, w, senders, rowptr, out);
    return after_launch();
}

int e3j_conv_bwd_f64(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const double* x, const double* sh,
                     const double* w, const int32_t* senders, const int32_t* receivers, const int32_t* sender_perm,
                     const int32_t* colptr, const double* grad_out, double* grad_x, double* grad_sh, double* grad_w,
                     void* workspace, size_t workspace_bytes, void* stream) {
    if (!basic_args_ok(plan, n_nodes, n_edges)) return E3J_ERR_INVALID_ARG;
    if (n_nodes == 0) return E3J_OK;
    if (!x || !grad_out || (n_edges > 0 && (!sh || !w || !senders || !receivers))) return E3J_ERR_INVALID_ARG;
    if ((sender_perm == nullptr) != (colptr == nullptr)) return E3J_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (grad_x && !sender_perm) {
        if (!workspace || ((uintptr_t)workspace & 255u) || workspace_bytes < e3j_conv_f64_workspace_bytes(plan, n_nodes, n_edges))
            return E3J_ERR_WORKSPACE;
        char* ws = (char*)workspace;
        const size_t sec = align_up(4 * (size_t)(n_nodes + 1), 256);
        int32_t* cp = (int32_t*)(ws + sec);
        int32_t* pm = (int32_t*)(ws + 2 * sec);
        if (int s = graph_prepare(n_nodes, n_edges, senders, receivers, nullptr, pm, cp, st)) return s;
        sender_perm = pm; colptr = cp;
    }
    DeviceTables t;
    if (int s = get_device_tables(plan, t)) return s;
    const Dims dm{plan->nq, plan->d, plan->dp, plan->P, plan->D, (plan->flags & E3J_PLAN_COLLAPSE_OUTPUTS) ? 1 : 0};
    if ((grad_w || grad_sh) && n_edges > 0) {
        bwd_edge_f64_kernel<<<grid_for(n_edges), 256, 0, st>>>(t, dm, n_edges, x, sh, w, senders, receivers, grad_out,
                                                              grad_w, grad_sh);
        if (int s = after_launch()) return s;
    }
    if (grad_x) {
        bwd_node_f64_kernel<<<grid_for(n_nodes), 256, 0, st>>>(t, dm, n_nodes, sh, w, receivers, sender_perm, colptr,
                                                              grad_out, grad_x);
        if (int s = after_launch()) return s;
    }
    return E3J_OK;
}

}  // extern "C"
