// Scheduled backward: entry points (the order is built on the host by bwd_schedule.cpp, the sweep is
// fast/fast_bwd1s.cuh).
#include <vector>

#include "bwd_schedule.hpp"
#include "common.cuh"
#include "fast_registry.hpp"

using namespace e3j;

namespace {

const FastKernels* sched_kernels(const e3j_plan* plan) {
    const FastKernels* fk = plan ? fast_lookup(plan) : nullptr;
    return (fk && fk->conv_bwd_sched && fk->sched_T > 0) ? fk : nullptr;
}

bool args_ok(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges) {
    return plan && n_nodes >= 0 && n_edges >= 0 && n_nodes < (1ll << 31) - 1 && n_edges < (1ll << 31) - 1;
}

}  // namespace

extern "C" {

size_t e3j_bwd_schedule_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges) {
    const FastKernels* fk = sched_kernels(plan);
    if (!fk || !args_ok(plan, n_nodes, n_edges)) return 0;
    return align_up(4 * bwd_schedule_max_words(fk->sched_T, sm_count(), n_nodes, n_edges), 256);
}

int e3j_bwd_schedule_build(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const int32_t* senders_host,
                           const int32_t* receivers_host, void* schedule_dev, size_t schedule_bytes, void* stream) {
    if (!args_ok(plan, n_nodes, n_edges)) return E3J_ERR_INVALID_ARG;
    const FastKernels* fk = sched_kernels(plan);
    if (!fk) return E3J_ERR_UNSUPPORTED;
    if (n_edges > 0 && (!senders_host || !receivers_host)) return E3J_ERR_INVALID_ARG;
    if (!schedule_dev || ((uintptr_t)schedule_dev & 255u)) return E3J_ERR_WORKSPACE;
    std::vector<int32_t> words;
    if (build_bwd_schedule(fk->sched_T, sm_count(), n_nodes, n_edges, senders_host, receivers_host, words))
        return E3J_ERR_INVALID_ARG;
    if (4 * words.size() > schedule_bytes) return E3J_ERR_WORKSPACE;
    // the host vector dies with this call: the copy must have left it before we return
    E3J_CUDA_TRY(cudaMemcpyAsync(schedule_dev, words.data(), 4 * words.size(), cudaMemcpyHostToDevice, (cudaStream_t)stream));
    E3J_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    return E3J_OK;
}

int e3j_conv_bwd_scheduled(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x, const float* sh,
                           const float* w, const void* schedule_dev, const float* grad_out, float* grad_x,
                           float* grad_sh, float* grad_w, void* workspace, size_t workspace_bytes, void* stream) {
    if (!args_ok(plan, n_nodes, n_edges)) return E3J_ERR_INVALID_ARG;
    const FastKernels* fk = sched_kernels(plan);
    if (!fk) return E3J_ERR_UNSUPPORTED;
    if (n_nodes == 0) return E3J_OK;
    if (!x || !grad_out || !grad_x || !schedule_dev) return E3J_ERR_INVALID_ARG;
    if (n_edges > 0 && (!sh || !w || !grad_sh || !grad_w)) return E3J_ERR_INVALID_ARG;
    if (((uintptr_t)x | (uintptr_t)w | (uintptr_t)grad_out | (uintptr_t)grad_x | (uintptr_t)grad_w | (uintptr_t)sh |
         (uintptr_t)schedule_dev) & 15u)
        return E3J_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255u) || workspace_bytes < e3j_conv_bwd_workspace_bytes(plan, n_nodes, n_edges))
        return E3J_ERR_WORKSPACE;
    DeviceTables t;
    if (int s = get_device_tables(plan, t)) return s;
    ConvArgs a{};
    a.n_nodes = n_nodes; a.n_edges = n_edges; a.x = x; a.sh = sh; a.w = w; a.grad_out = grad_out;
    a.grad_x = grad_x; a.grad_sh = grad_sh; a.grad_w = grad_w;
    a.workspace = workspace; a.workspace_bytes = workspace_bytes; a.stream = (cudaStream_t)stream; a.status = t.status;
    return fk->conv_bwd_sched(a, (const int32_t*)schedule_dev);
}

}  // extern "C"
