// Internal helpers shared by the CUDA translation units of libe3j.
#pragma once
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

#include "plan.hpp"

namespace e3j {

extern thread_local int g_last_cuda_error;
extern std::atomic<int64_t> g_launch_count;

inline int cuda_status(cudaError_t err) {
    if (err == cudaSuccess) return E3J_OK;
    g_last_cuda_error = (int)err;
    return E3J_ERR_CUDA;
}

#define E3J_CUDA_TRY(expr)                                   \
    do {                                                     \
        const int _st = ::e3j::cuda_status((expr));          \
        if (_st != E3J_OK) return _st;                       \
    } while (0)

// Call after every kernel launch: counts it and converts a launch error to a status.
inline int after_launch() {
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return cuda_status(cudaGetLastError());
}

// Launch of a kernel that follows another one on the same stream and starts with fast::grid_dependency_wait(): the
// launch itself (and the scheduling of its first CTAs) overlaps the tail of its predecessor; the wait inside the
// kernel holds it until the predecessor has finished and its writes are visible (programmatic dependent launch).
template <class... KArgs, class... Args>
inline int launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return cuda_status(err != cudaSuccess ? err : cudaGetLastError());
}
// Device tables of `plan` on the current device (uploaded on first use).
int get_device_tables(const e3j_plan* plan, DeviceTables& out);

struct Dims {
    int nq, d, dp, P, D;
    int collapsed;  // several paths may share an output row (E3J_PLAN_COLLAPSE_OUTPUTS)
};

// Scalar description of a graph launch shared by the generic and specialised paths.
struct ConvArgs {
    int64_t n_nodes, n_edges;
    const float *x, *sh, *w;
    const int32_t *senders, *receivers, *rowptr, *sender_perm, *colptr;
    const float* grad_out;
    float *out, *grad_x, *grad_sh, *grad_w;
    void* workspace;
    size_t workspace_bytes;
    cudaStream_t stream;
    int32_t* status;  // device status word of the plan on this device
    const int32_t* n_real;  // padded call: device word with the number of real edges (rowptr[n_nodes]); else null
    const float* vec;       // forward: edge vectors [E][3] in place of sh (the kernel forms the harmonics); else null
};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// SM count of the current device (cached per thread; grids are sized in multiples of it), capped at kMaxSms,
// the bound that scratch sizes are computed with.  148 (B200) if the device cannot be queried.
constexpr int kMaxSms = 192;
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

// The bodies of e3j_conv_fwd / e3j_conv_bwd (and their padded forms), for entry points that compose them.
int conv_fwd_impl(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x, const float* sh,
                  const float* w, const int32_t* senders, const int32_t* receivers, const int32_t* rowptr,
                  float* out, void* workspace, size_t workspace_bytes, void* stream, bool padded,
                  const float* edge_vec = nullptr);   // edge_vec: specialised kernels only, in place of sh
// Harmonics of edge vectors (harmonics.cu): sh [n, (lmax+1)^2] from vec [n, 3] and the gradient back; lmax <= 3.
int harmonics_fwd(int lmax, int64_t n, const float* vec, float* sh, cudaStream_t st);
int harmonics_bwd(int lmax, int64_t n, const float* vec, const float* grad_sh, float* grad_vec, cudaStream_t st);
int plan_sh_lmax(const e3j_plan* plan);   // lmax of the plan's harmonics if they are the full set l <= 3, else -1
// Does the plan run on signature-specialised kernels (which can form the harmonics from edge vectors themselves)?
bool has_fast_forward(const e3j_plan* plan);
int conv_bwd_impl(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x, const float* sh,
                  const float* w, const int32_t* senders, const int32_t* receivers, const int32_t* rowptr,
                  const int32_t* sender_perm, const int32_t* colptr, const float* grad_out, float* grad_x,
                  float* grad_sh, float* grad_w, void* workspace, size_t workspace_bytes, void* stream, bool padded);

}  // namespace e3j
