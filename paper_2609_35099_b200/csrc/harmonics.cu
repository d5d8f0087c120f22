// Harmonics of the edge vectors (paper, "Key Operations in Scope": the harmonic embedding of the edge direction),
// as kernels of their own and composed with the convolution.
//
//   e3j_harmonics_fwd / _bwd   sh = Y(vec / |vec|), grad_vec = (dY/dvec)^T grad_sh; one thread per edge
//   e3j_conv_vec_fwd           the forward convolution on edge vectors: the specialised kernels form the harmonics
//                              in their table warp (no [E, d'] array is read or written); plans on the table-driven
//                              kernels get them from e3j_harmonics_fwd through the workspace
//   e3j_conv_vec_bwd           composed: harmonics into the workspace, e3j_conv_bwd with grad_sh kept as scratch,
//                              then the chain rule into the vectors
#include "common.cuh"
#include "fast/harmonics.cuh"

namespace e3j {
namespace {

template <int DSH>
__global__ void __launch_bounds__(256)
harmonics_fwd_kernel(int64_t n, const float* __restrict__ vec, float* __restrict__ sh) {
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) {
        float x, y, z, inv_r, Y[DSH];
        fast::unit_vector(vec[3 * e], vec[3 * e + 1], vec[3 * e + 2], x, y, z, inv_r);
        fast::harmonics<DSH>(x, y, z, Y);
        if constexpr (DSH % 4 == 0) {   // a row is a whole number of 16-byte pieces (cudaMalloc'ed arrays are aligned)
            float4* row = reinterpret_cast<float4*>(sh + e * DSH);
#pragma unroll
            for (int i = 0; i < DSH / 4; ++i) row[i] = make_float4(Y[4 * i], Y[4 * i + 1], Y[4 * i + 2], Y[4 * i + 3]);
        } else {
#pragma unroll
            for (int i = 0; i < DSH; ++i) sh[e * DSH + i] = Y[i];
        }
    }
}

// grad_vec = (I - u u^T) / r * sum_i grad_sh_i grad Y_i(u): Y is a function of the direction only
template <int DSH>
__global__ void __launch_bounds__(256)
harmonics_bwd_kernel(int64_t n, const float* __restrict__ vec, const float* __restrict__ grad_sh,
                     float* __restrict__ grad_vec) {
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) {
        float x, y, z, inv_r, g[DSH], gx, gy, gz;
        fast::unit_vector(vec[3 * e], vec[3 * e + 1], vec[3 * e + 2], x, y, z, inv_r);
        if constexpr (DSH % 4 == 0) {
            const float4* row = reinterpret_cast<const float4*>(grad_sh + e * DSH);
#pragma unroll
            for (int i = 0; i < DSH / 4; ++i) {
                const float4 v = row[i];
                g[4 * i] = v.x; g[4 * i + 1] = v.y; g[4 * i + 2] = v.z; g[4 * i + 3] = v.w;
            }
        } else {
#pragma unroll
            for (int i = 0; i < DSH; ++i) g[i] = grad_sh[e * DSH + i];
        }
        fast::harmonics_vjp<DSH>(x, y, z, g, gx, gy, gz);
        const float radial = fmaf(gx, x, fmaf(gy, y, gz * z));
        grad_vec[3 * e] = (gx - radial * x) * inv_r;
        grad_vec[3 * e + 1] = (gy - radial * y) * inv_r;
        grad_vec[3 * e + 2] = (gz - radial * z) * inv_r;
    }
}

inline int grid_for(int64_t n) { return (int)std::min<int64_t>((n + 255) / 256, (int64_t)sm_count() * 16); }

}  // namespace

int harmonics_fwd(int lmax, int64_t n, const float* vec, float* sh, cudaStream_t st) {
    if (n == 0) return E3J_OK;
    switch (lmax) {
        case 0: harmonics_fwd_kernel<1><<<grid_for(n), 256, 0, st>>>(n, vec, sh); break;
        case 1: harmonics_fwd_kernel<4><<<grid_for(n), 256, 0, st>>>(n, vec, sh); break;
        case 2: harmonics_fwd_kernel<9><<<grid_for(n), 256, 0, st>>>(n, vec, sh); break;
        case 3: harmonics_fwd_kernel<16><<<grid_for(n), 256, 0, st>>>(n, vec, sh); break;
        default: return E3J_ERR_UNSUPPORTED;
    }
    return after_launch();
}

int harmonics_bwd(int lmax, int64_t n, const float* vec, const float* grad_sh, float* grad_vec, cudaStream_t st) {
    if (n == 0) return E3J_OK;
    switch (lmax) {
        case 0: harmonics_bwd_kernel<1><<<grid_for(n), 256, 0, st>>>(n, vec, grad_sh, grad_vec); break;
        case 1: harmonics_bwd_kernel<4><<<grid_for(n), 256, 0, st>>>(n, vec, grad_sh, grad_vec); break;
        case 2: harmonics_bwd_kernel<9><<<grid_for(n), 256, 0, st>>>(n, vec, grad_sh, grad_vec); break;
        case 3: harmonics_bwd_kernel<16><<<grid_for(n), 256, 0, st>>>(n, vec, grad_sh, grad_vec); break;
        default: return E3J_ERR_UNSUPPORTED;
    }
    return after_launch();
}

// lmax of the plan's harmonics, or -1 if d' is not (lmax + 1)^2 with lmax <= 3
int plan_sh_lmax(const e3j_plan* plan) {
    for (int l = 0; l <= 3; ++l)
        if ((l + 1) * (l + 1) == plan->dp) return l;
    return -1;
}

namespace {

// workspace of the calls on edge vectors: [convolution workspace | sh | grad_sh]
struct VecLayout { size_t conv, conv_bytes, sh, gsh, total; };
VecLayout vec_layout(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, bool bwd) {
    VecLayout L{};
    L.conv_bytes = bwd ? e3j_conv_bwd_workspace_bytes(plan, n_nodes, n_edges)
                       : e3j_conv_fwd_workspace_bytes(plan, n_nodes, n_edges);
    const size_t sh_bytes = align_up(4 * (size_t)std::max<int64_t>(n_edges, 1) * plan->dp, 256);
    size_t off = align_up(L.conv_bytes, 256);
    L.sh = off; if (bwd || !has_fast_forward(plan)) off += sh_bytes;
    L.gsh = off; if (bwd) off += sh_bytes;
    L.total = off;
    return L;
}

bool args_ok(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges) {
    return plan && n_nodes >= 0 && n_edges >= 0 && n_nodes < (1ll << 31) - 1 && n_edges < (1ll << 31) - 1;
}

}  // namespace
}  // namespace e3j

using namespace e3j;

extern "C" {

int e3j_harmonics_fwd(int lmax, int64_t n_edges, const float* edge_vec, float* sh, void* stream) {
    if (n_edges < 0 || lmax < 0) return E3J_ERR_INVALID_ARG;
    if (n_edges > 0 && (!edge_vec || !sh)) return E3J_ERR_INVALID_ARG;
    if ((uintptr_t)sh & 15u) return E3J_ERR_INVALID_ARG;
    return harmonics_fwd(lmax, n_edges, edge_vec, sh, (cudaStream_t)stream);
}

int e3j_harmonics_bwd(int lmax, int64_t n_edges, const float* edge_vec, const float* grad_sh, float* grad_vec,
                      void* stream) {
    if (n_edges < 0 || lmax < 0) return E3J_ERR_INVALID_ARG;
    if (n_edges > 0 && (!edge_vec || !grad_sh || !grad_vec)) return E3J_ERR_INVALID_ARG;
    if ((uintptr_t)grad_sh & 15u) return E3J_ERR_INVALID_ARG;
    return harmonics_bwd(lmax, n_edges, edge_vec, grad_sh, grad_vec, (cudaStream_t)stream);
}

size_t e3j_conv_vec_fwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges) {
    if (!args_ok(plan, n_nodes, n_edges)) return 0;
    return vec_layout(plan, n_nodes, n_edges, false).total;
}

size_t e3j_conv_vec_bwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges) {
    if (!args_ok(plan, n_nodes, n_edges)) return 0;
    return vec_layout(plan, n_nodes, n_edges, true).total;
}

int e3j_conv_vec_fwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x, const float* edge_vec,
                     const float* w, const int32_t* senders, const int32_t* receivers, const int32_t* rowptr,
                     float* out, void* workspace, size_t workspace_bytes, void* stream) {
    if (!args_ok(plan, n_nodes, n_edges)) return E3J_ERR_INVALID_ARG;
    const int lmax = plan_sh_lmax(plan);
    if (lmax < 0) return E3J_ERR_UNSUPPORTED;
    if (n_edges > 0 && !edge_vec) return E3J_ERR_INVALID_ARG;
    const VecLayout L = vec_layout(plan, n_nodes, n_edges, false);
    if (!workspace || ((uintptr_t)workspace & 255u) || workspace_bytes < L.total) return E3J_ERR_WORKSPACE;
    char* ws = (char*)workspace;
    if (has_fast_forward(plan))
        return conv_fwd_impl(plan, n_nodes, n_edges, x, nullptr, w, senders, receivers, rowptr, out, ws + L.conv,
                             L.conv_bytes, stream, false, edge_vec);
    float* sh = (float*)(ws + L.sh);
    if (int rc = harmonics_fwd(lmax, n_edges, edge_vec, sh, (cudaStream_t)stream)) return rc;
    return conv_fwd_impl(plan, n_nodes, n_edges, x, sh, w, senders, receivers, rowptr, out, ws + L.conv, L.conv_bytes,
                         stream, false);
}

int e3j_conv_vec_bwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x, const float* edge_vec,
                     const float* w, const int32_t* senders, const int32_t* receivers, const int32_t* rowptr,
                     const int32_t* sender_perm, const int32_t* colptr, const float* grad_out, float* grad_x,
                     float* grad_vec, float* grad_w, void* workspace, size_t workspace_bytes, void* stream) {
    if (!args_ok(plan, n_nodes, n_edges)) return E3J_ERR_INVALID_ARG;
    const int lmax = plan_sh_lmax(plan);
    if (lmax < 0) return E3J_ERR_UNSUPPORTED;
    if (n_edges > 0 && !edge_vec) return E3J_ERR_INVALID_ARG;
    const VecLayout L = vec_layout(plan, n_nodes, n_edges, true);
    if (!workspace || ((uintptr_t)workspace & 255u) || workspace_bytes < L.total) return E3J_ERR_WORKSPACE;
    char* ws = (char*)workspace;
    cudaStream_t st = (cudaStream_t)stream;
    float* sh = (float*)(ws + L.sh);
    float* gsh = (float*)(ws + L.gsh);
    if (int rc = harmonics_fwd(lmax, n_edges, edge_vec, sh, st)) return rc;
    if (int rc = conv_bwd_impl(plan, n_nodes, n_edges, x, sh, w, senders, receivers, rowptr, sender_perm, colptr,
                               grad_out, grad_x, grad_vec ? gsh : nullptr, grad_w, ws + L.conv, L.conv_bytes, stream,
                               false)) return rc;
    if (grad_vec && n_nodes > 0)
        if (int rc = harmonics_bwd(lmax, n_edges, edge_vec, gsh, grad_vec, st)) return rc;
    return E3J_OK;
}

}  // extern "C"
