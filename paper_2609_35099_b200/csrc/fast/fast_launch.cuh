// Host-side launchers of the signature-specialised kernels.
#pragma once
#include "../fast_registry.hpp"
#include "fast_fwd.cuh"

namespace e3j {
namespace fast {

constexpr int kMaxSms = 192;       // upper bound on the SM count, for scratch sizing
constexpr size_t kPartRecvBytes = 8192;  // slot of the [n_cta][2] boundary receiver ids

inline int sm_count() {
    static thread_local int cached_dev = -1, cached = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (dev != cached_dev) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached = n > kMaxSms ? kMaxSms : n;
        cached_dev = dev;
    }
    return cached;
}

// scratch: [part_recv: 2*n_cta ints in an 8 KB slot][partial rows: 2*n_cta*D*NQ floats], n_cta <= kMaxSms*S::FC
template <class S>
size_t fwd_scratch_bytes(int64_t, int64_t) {
    return kPartRecvBytes + sizeof(float) * 2 * (size_t)kMaxSms * S::FC * S::D * S::NQ;
}

template <class S>
int launch_fwd(const ConvArgs& a) {
    using L = FwdSmem<S>;
    static_assert(L::total * S::FC + 1024 * S::FC <= 228 * 1024, "forward stage ring does not fit in shared memory");
    static_assert(2 * kMaxSms * S::FC * sizeof(int32_t) <= kPartRecvBytes, "part_recv does not fit its slot");
    if (a.workspace_bytes < fwd_scratch_bytes<S>(a.n_nodes, a.n_edges)) return E3J_ERR_WORKSPACE;
    const int n_cta = sm_count() * S::FC;
    static thread_local int attr_dev = -1;
    int dev = 0;
    E3J_CUDA_TRY(cudaGetDevice(&dev));
    if (attr_dev != dev) {
        E3J_CUDA_TRY(cudaFuncSetAttribute(fast_fwd_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::total));
        attr_dev = dev;
    }
    FwdParams p{};
    p.x = a.x; p.sh = a.sh; p.w = a.w; p.senders = a.senders; p.receivers = a.receivers; p.out = a.out;
    p.n_nodes = a.n_nodes; p.n_edges = a.n_edges;
    const int64_t per = (a.n_edges + n_cta - 1) / n_cta;
    p.chunk = (per + 3) / 4 * 4;
    p.part_recv = reinterpret_cast<int32_t*>(a.workspace);
    p.partial = reinterpret_cast<float*>(reinterpret_cast<char*>(a.workspace) + kPartRecvBytes);
    p.status = a.status;
    constexpr int threads = (S::FW * (S::NQ / (32 * S::V)) + 1) * 32;  // consumers + one producer warp
    fast_fwd_kernel<S><<<n_cta, threads, L::total, a.stream>>>(p);
    if (int s = after_launch()) return s;
    fwd_fixup_kernel<<<n_cta, 256, 0, a.stream>>>(n_cta, S::D * S::NQ / 4, reinterpret_cast<const float4*>(p.partial),
                                                 p.part_recv, reinterpret_cast<float4*>(a.out));
    return after_launch();
}

}  // namespace fast
}  // namespace e3j

#ifdef E3J_PROF
// debug builds only: copies the forward kernel's cycle counters to the host
extern "C" __attribute__((weak)) int e3j_debug_fwd_prof(long long* host, int n) {
    return (int)cudaMemcpyFromSymbol(host, e3j::fast::g_fwd_prof, sizeof(long long) * n);
}
#endif
