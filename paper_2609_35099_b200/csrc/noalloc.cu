// Forward convolution for callers that cannot allocate device memory.
//
// The specialised forward kernel needs scratch for the receiver rows that straddle two CTAs'
// edge ranges.  e3j_conv_fwd takes that scratch from a caller-provided workspace; the entry
// point below keeps it in a file-scope __device__ array instead, so the caller passes inputs and
// the output only and nothing here (or below) calls cudaMalloc / cudaFree or any allocating
// library routine.  Every GPU that loads the library holds the array until the process exits.
#include <mutex>

#include "common.cuh"
#include "fast_registry.hpp"

#define E3J_NOALLOC_SCRATCH_BYTES (24u << 20) /* 24 MiB; see e3j.h */

namespace {

// In host code this name is only a handle for the runtime's symbol table, not a device address:
// the address is fetched with cudaGetSymbolAddress, once per device, with that device current.
static __device__ __align__(256) unsigned char g_noalloc_scratch[E3J_NOALLOC_SCRATCH_BYTES];

// Status word of the kernels launched from here (0 = fine, non-zero = a bounded wait gave up and the output is
// invalid): file scope for the same reason as the scratch, read and cleared by e3j_noalloc_status.
static __device__ int32_t g_noalloc_status;

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {nullptr};
int32_t* g_status_ptr[kMaxDevices] = {nullptr};

int scratch_for_current_device(void** out, int32_t** status) {
    int dev = 0;
    E3J_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return E3J_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[dev]) {
        void* ptr = nullptr;
        void* st = nullptr;
        E3J_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
        E3J_CUDA_TRY(cudaGetSymbolAddress(&st, g_noalloc_status));
        if (!ptr || !st || (reinterpret_cast<uintptr_t>(ptr) & 255u)) return E3J_ERR_WORKSPACE;
        g_status_ptr[dev] = static_cast<int32_t*>(st);   // zero-initialised with the module
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    *status = g_status_ptr[dev];
    return E3J_OK;
}

}  // namespace

extern "C" int e3j_conv_fwd_noalloc(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x,
                                    const float* sh, const float* w, const int32_t* senders,
                                    const int32_t* receivers, float* out, void* stream) {
    using namespace e3j;
    if (!plan || n_nodes < 0 || n_edges < 0 || n_nodes >= (1ll << 31) - 1 || n_edges >= (1ll << 31) - 1)
        return E3J_ERR_INVALID_ARG;
    if (n_nodes == 0) return E3J_OK;
    if (!out || !x) return E3J_ERR_INVALID_ARG;
    if (n_edges > 0 && (!sh || !w || !senders || !receivers)) return E3J_ERR_INVALID_ARG;
    if (((uintptr_t)x | (uintptr_t)w | (uintptr_t)out) & 15u) return E3J_ERR_INVALID_ARG;  // 128-bit rows
    const FastKernels* fk = fast_lookup(plan);
    if (!fk || !fk->conv_fwd || !fk->fwd_scratch_bytes) return E3J_ERR_UNSUPPORTED;  // no specialised kernel
    cudaStream_t st = (cudaStream_t)stream;
    if (n_edges == 0) {  // every receiver row is empty
        E3J_CUDA_TRY(cudaMemsetAsync(out, 0, sizeof(float) * (size_t)n_nodes * plan->D * plan->nq, st));
        return E3J_OK;
    }
    // the need depends on the plan (D * N_q) and on the SM count of the current device, not on the graph
    if (fk->fwd_scratch_bytes(n_nodes, n_edges) > (size_t)E3J_NOALLOC_SCRATCH_BYTES) return E3J_ERR_WORKSPACE;
    void* scratch = nullptr;
    int32_t* status = nullptr;
    if (int s = scratch_for_current_device(&scratch, &status)) return s;
    ConvArgs a{};
    a.n_nodes = n_nodes; a.n_edges = n_edges; a.x = x; a.sh = sh; a.w = w;
    a.senders = senders; a.receivers = receivers; a.out = out;
    a.workspace = scratch; a.workspace_bytes = E3J_NOALLOC_SCRATCH_BYTES; a.stream = st;
    a.status = status;   // the plan's own status word lives in allocated memory; this one does not
    // nothing in the scratch has to start at zero: the kernel writes every word it later reads
    return fk->conv_fwd(a);
}


extern "C" int e3j_noalloc_status(int32_t* status) {
    using namespace e3j;
    if (!status) return E3J_ERR_INVALID_ARG;
    void* scratch = nullptr;
    int32_t* word = nullptr;
    if (int s = scratch_for_current_device(&scratch, &word)) return s;
    E3J_CUDA_TRY(cudaDeviceSynchronize());
    E3J_CUDA_TRY(cudaMemcpy(status, word, sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (*status != 0) E3J_CUDA_TRY(cudaMemset(word, 0, sizeof(int32_t)));
    return E3J_OK;
}
