// Host-side launchers of the signature-specialised kernels.
#pragma once
#include <algorithm>

#include "../fast_registry.hpp"
#include "fast_bwd.cuh"
#include "fast_bwd1.cuh"
#include "fast_fwd.cuh"

namespace e3j {
namespace fast {

using e3j::kMaxSms;   // upper bound on the SM count, for scratch sizing
using e3j::sm_count;
constexpr size_t kPartRecvBytes = 8192;  // slot of the [n_cta][2] boundary receiver ids

// scratch: [part_recv: 2*n_cta ints in an 8 KB slot][partial rows: 2*n_cta*D*NQ floats],
// n_cta = (SMs of the current device) * S::FC
template <class S>
size_t fwd_scratch_need(int n_cta) {
    return kPartRecvBytes + sizeof(float) * 2 * (size_t)n_cta * S::D * S::NQ;
}
template <class S>
size_t fwd_scratch_bytes(int64_t, int64_t) {
    return fwd_scratch_need<S>(sm_count() * S::FC);
}

template <class S>
int launch_fwd(const ConvArgs& a) {
    using L = FwdSmem<S>;
    static_assert(L::total * S::FC + 1024 * S::FC <= 228 * 1024, "forward stage ring does not fit in shared memory");
    static_assert(2 * kMaxSms * S::FC * sizeof(int32_t) <= kPartRecvBytes, "part_recv does not fit its slot");
    const int n_cta = sm_count() * S::FC;
    if (a.workspace_bytes < fwd_scratch_need<S>(n_cta)) return E3J_ERR_WORKSPACE;
    static thread_local int attr_dev = -1;
    int dev = 0;
    E3J_CUDA_TRY(cudaGetDevice(&dev));
    if (attr_dev != dev) {
        E3J_CUDA_TRY(cudaFuncSetAttribute(fast_fwd_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::total));
        attr_dev = dev;
    }
    FwdParams p{};
    p.x = a.x; p.sh = a.sh; p.w = a.w; p.senders = a.senders; p.receivers = a.receivers; p.out = a.out;
    p.vec = a.vec;
    p.n_nodes = a.n_nodes; p.n_edges = a.n_edges;
    const int64_t per = (a.n_edges + n_cta - 1) / n_cta;
    p.chunk = (per + 3) / 4 * 4;
    p.part_recv = reinterpret_cast<int32_t*>(a.workspace);
    p.partial = reinterpret_cast<float*>(reinterpret_cast<char*>(a.workspace) + kPartRecvBytes);
    p.status = a.status;
    p.n_real = a.n_real;
    constexpr int threads = (S::FW * (S::NQ / (32 * S::V)) + 2) * 32;  // consumers + two producer warps
    fast_fwd_kernel<S><<<n_cta, threads, L::total, a.stream>>>(p);
    if (int s = after_launch()) return s;
    return launch_dependent(fwd_fixup_kernel, dim3(n_cta), dim3(256), 0, a.stream, n_cta, S::D * S::NQ / 4, reinterpret_cast<const float4*>(p.partial),
                                                 p.part_recv, reinterpret_cast<float4*>(a.out));
}

// Standalone tensor product = the forward kernel with every row its own sender and receiver: no row
// straddles a CTA boundary, so there is no scratch and no fix-up launch.
template <class S>
int launch_tp_fwd(int64_t rows, const float* x1, const float* x2, const float* w, float* out, cudaStream_t st) {
    using L = FwdSmem<S>;
    const int n_cta = sm_count() * S::FC;
    static thread_local int attr_dev = -1;
    int dev = 0;
    E3J_CUDA_TRY(cudaGetDevice(&dev));
    if (attr_dev != dev) {
        E3J_CUDA_TRY(cudaFuncSetAttribute(fast_fwd_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::total));
        attr_dev = dev;
    }
    FwdParams p{};
    p.x = x1; p.sh = x2; p.w = w; p.out = out; p.n_nodes = rows; p.n_edges = rows; p.identity = 1;
    const int64_t per = (rows + n_cta - 1) / n_cta;
    p.chunk = (per + 3) / 4 * 4;
    constexpr int threads = (S::FW * (S::NQ / (32 * S::V)) + 2) * 32;
    fast_fwd_kernel<S><<<n_cta, threads, L::total, st>>>(p);
    return after_launch();
}

template <class S>
int launch_tp_bwd(int64_t rows, const float* x1, const float* x2, const float* w, const float* g, float* gx1,
                  float* gx2, float* gw, cudaStream_t st) {
    using L = BwdSmem<S>;
    if (!gx1) return E3J_ERR_UNSUPPORTED;  // (the row's share of grad_x1 is stored unconditionally) caller falls back to the generic kernels
    constexpr bool kRowwise = S::ETR > 0;   // one warp per row, one CTA per SM (fast_bwd1.cuh)
    const int n_cta = sm_count() * (kRowwise ? 1 : S::BC);
    BwdParams p{};
    p.x = x1; p.sh = x2; p.w = w; p.grad_out = g; p.grad_sh = gx2; p.grad_w = gw;
    p.dx_edge = gx1;  // each row is its own sender: the per-edge share is the gradient
    p.n_nodes = rows; p.n_edges = rows; p.identity = 1;
    p.chunk = (rows + n_cta - 1) / n_cta;
    static thread_local int attr_dev = -1;
    int dev = 0;
    E3J_CUDA_TRY(cudaGetDevice(&dev));
    if constexpr (kRowwise) {
        using L1 = Bwd1Smem<S, true>;
        static_assert(L1::total + 1024 <= 228 * 1024, "row-wise backward ring does not fit in shared memory");
        if (attr_dev != dev) {
            E3J_CUDA_TRY(cudaFuncSetAttribute(fast_bwd1_kernel<S, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L1::total));
            attr_dev = dev;
        }
        fast_bwd1_kernel<S, true><<<n_cta, (L1::T * L1::CH * L1::NG + 1) * 32, L1::total, st>>>(p);
    } else {
        if (attr_dev != dev) {
            E3J_CUDA_TRY(cudaFuncSetAttribute(fast_bwd_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::total));
            attr_dev = dev;
        }
        constexpr int threads = (S::BW * (S::NQ / (32 * S::BV)) + 1) * 32;  // consumers + one producer warp
        fast_bwd_kernel<S><<<n_cta, threads, L::total, st>>>(p);
    }
    return after_launch();
}

// scratch of the backward: this edge's share of grad_x, [E][d][N_q]
template <class S>
size_t bwd_scratch_bytes(int64_t, int64_t n_edges) {
    return align_up(sizeof(float) * (size_t)(n_edges > 0 ? n_edges : 1) * S::DIN * S::NQ, 256);
}

template <class S>
int launch_bwd(const ConvArgs& a) {
    using L = BwdSmem<S>;
    static_assert(L::total * S::BC + 1024 * S::BC <= 228 * 1024, "backward stage ring does not fit in shared memory");
    if (a.workspace_bytes < bwd_scratch_bytes<S>(a.n_nodes, a.n_edges)) return E3J_ERR_WORKSPACE;
    constexpr bool kEdgewise = S::ET > 0;   // one warp per edge, one CTA per SM (fast_bwd1.cuh)
    const int n_cta = sm_count() * (kEdgewise ? 1 : S::BC);
    BwdParams p{};
    p.x = a.x; p.sh = a.sh; p.w = a.w; p.senders = a.senders; p.receivers = a.receivers;
    p.grad_out = a.grad_out; p.grad_sh = a.grad_sh; p.grad_w = a.grad_w;
    p.dx_edge = reinterpret_cast<float*>(a.workspace);
    p.n_nodes = a.n_nodes; p.n_edges = a.n_edges;
    p.chunk = (a.n_edges + n_cta - 1) / n_cta;
    p.status = a.status;
    p.n_real = a.n_real;
    static thread_local int attr_dev = -1;
    int dev = 0;
    E3J_CUDA_TRY(cudaGetDevice(&dev));
    if constexpr (kEdgewise) {
        using L1 = Bwd1Smem<S, false>;
        static_assert(L1::total + 1024 <= 228 * 1024, "edge-wise backward ring does not fit in shared memory");
        if (attr_dev != dev) {
            E3J_CUDA_TRY(cudaFuncSetAttribute(fast_bwd1_kernel<S, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L1::total));
            attr_dev = dev;
        }
        fast_bwd1_kernel<S, false><<<n_cta, (L1::T * L1::CH + 1) * 32, L1::total, a.stream>>>(p);  // consumers + one producer warp
    } else {
        if (attr_dev != dev) {
            E3J_CUDA_TRY(cudaFuncSetAttribute(fast_bwd_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::total));
            attr_dev = dev;
        }
        constexpr int threads = (S::BW * (S::NQ / (32 * S::BV)) + 1) * 32;  // consumers + one producer warp
        fast_bwd_kernel<S><<<n_cta, threads, L::total, a.stream>>>(p);
    }
    if (int s = after_launch()) return s;
    if (a.n_real) {
        bwd_zero_padding_kernel<<<sm_count() * 8, 256, 0, a.stream>>>(a.n_real, a.n_edges, S::P * S::NQ / 4, S::DSH,
                                                              reinterpret_cast<float4*>(a.grad_w), a.grad_sh);
        if (int s = after_launch()) return s;
    }
    if (!a.grad_x) return E3J_OK;   // the shares stay in the scratch
    // one CTA per sender: the hardware hands them out as CTAs finish, so uneven degrees do not leave a tail
    const int64_t blocks = std::min<int64_t>(a.n_nodes, (int64_t)1 << 30);
    return launch_dependent(bwd_dx_reduce_kernel, dim3((int)blocks), dim3(S::DIN * S::NQ / 4), 0, a.stream, a.n_nodes, S::DIN * S::NQ / 4,
        reinterpret_cast<const float4*>(p.dx_edge), a.sender_perm, a.colptr, reinterpret_cast<float4*>(a.grad_x));
}

// Fused double backward, edge outputs: the edge-wise sweep over (x, sh, w) and their cotangents, then the
// sender-ordered sum of the per-edge shares (the scratch is that of launch_bwd).
template <class S>
int launch_dbl_edges(const ConvArgs& a, const float* ct_x, const float* ct_sh, const float* ct_w) {
    using L1 = Bwd1Smem<S, false, true>;
    static_assert(L1::total + 1024 <= 228 * 1024, "double-backward ring does not fit in shared memory");
    static_assert(L1::T < 30, "lanes 30 and 31 of the producer issue the tile's shared copies");
    if (a.workspace_bytes < bwd_scratch_bytes<S>(a.n_nodes, a.n_edges)) return E3J_ERR_WORKSPACE;
    const int n_cta = sm_count();
    BwdParams p{};
    p.x = a.x; p.sh = a.sh; p.w = a.w; p.senders = a.senders; p.receivers = a.receivers;
    p.ct_x = ct_x; p.ct_sh = ct_sh; p.ct_w = ct_w;
    p.grad_out = a.grad_out; p.grad_sh = a.grad_sh; p.grad_w = a.grad_w;
    p.dx_edge = reinterpret_cast<float*>(a.workspace);
    p.n_nodes = a.n_nodes; p.n_edges = a.n_edges;
    p.chunk = (a.n_edges + n_cta - 1) / n_cta;
    p.status = a.status;
    static thread_local int attr_dev = -1;
    int dev = 0;
    E3J_CUDA_TRY(cudaGetDevice(&dev));
    if (attr_dev != dev) {
        E3J_CUDA_TRY(cudaFuncSetAttribute(fast_bwd1_kernel<S, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L1::total));
        attr_dev = dev;
    }
    fast_bwd1_kernel<S, false, true><<<n_cta, (L1::T * L1::CH + 1) * 32, L1::total, a.stream>>>(p);
    if (int s = after_launch()) return s;
    const int64_t blocks = std::min<int64_t>(a.n_nodes, (int64_t)1 << 30);
    return launch_dependent(bwd_dx_reduce_kernel, dim3((int)blocks), dim3(S::DIN * S::NQ / 4), 0, a.stream, a.n_nodes, S::DIN * S::NQ / 4,
        reinterpret_cast<const float4*>(p.dx_edge), a.sender_perm, a.colptr, reinterpret_cast<float4*>(a.grad_x));
}

// Fused double backward, cotangent of grad_out: the forward sweep with two terms per coefficient pair, written
// to a.out (scratch and fix-up as in launch_fwd).
template <class S>
int launch_dbl_out(const ConvArgs& a, const float* ct_x, const float* ct_sh, const float* ct_w) {
    using L = FwdSmem<S, true>;
    static_assert(L::total * S::DFC + 1024 * S::DFC <= 228 * 1024, "double-backward forward ring does not fit in shared memory");
    static_assert(S::DFC <= S::FC, "the scratch is sized for the forward's CTA count");
    static_assert(L::T < 31, "lane 31 of the copy warp issues the tile's second weight copy");
    const int n_cta = sm_count() * S::DFC;
    if (a.workspace_bytes < fwd_scratch_need<S>(n_cta)) return E3J_ERR_WORKSPACE;
    static thread_local int attr_dev = -1;
    int dev = 0;
    E3J_CUDA_TRY(cudaGetDevice(&dev));
    if (attr_dev != dev) {
        E3J_CUDA_TRY(cudaFuncSetAttribute(fast_fwd_kernel<S, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::total));
        attr_dev = dev;
    }
    FwdParams p{};
    p.x = a.x; p.sh = a.sh; p.w = a.w; p.senders = a.senders; p.receivers = a.receivers; p.out = a.out;
    p.ct_x = ct_x; p.ct_sh = ct_sh; p.ct_w = ct_w;
    p.n_nodes = a.n_nodes; p.n_edges = a.n_edges;
    const int64_t per = (a.n_edges + n_cta - 1) / n_cta;
    p.chunk = (per + 3) / 4 * 4;
    p.part_recv = reinterpret_cast<int32_t*>(a.workspace);
    p.partial = reinterpret_cast<float*>(reinterpret_cast<char*>(a.workspace) + kPartRecvBytes);
    p.status = a.status;
    constexpr int threads = (L::NCONS + 2) * 32;  // consumers + two producer warps
    fast_fwd_kernel<S, true><<<n_cta, threads, L::total, a.stream>>>(p);
    if (int s = after_launch()) return s;
    return launch_dependent(fwd_fixup_kernel, dim3(n_cta), dim3(256), 0, a.stream, n_cta, S::D * S::NQ / 4, reinterpret_cast<const float4*>(p.partial),
                                                 p.part_recv, reinterpret_cast<float4*>(a.out));
}

}  // namespace fast
}  // namespace e3j
