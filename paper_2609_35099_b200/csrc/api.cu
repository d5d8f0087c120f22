// C ABI of libe3j: argument checking, device-table upload, kernel dispatch.
#include <algorithm>
#include <cstring>
#include <initializer_list>
#include <new>

#include "common.cuh"
#include "fast_registry.hpp"
#include "fast/fast_common.cuh"
#include "generic_kernels.cuh"

namespace e3j {

thread_local int g_last_cuda_error = 0;
std::atomic<int64_t> g_launch_count{0};

int graph_prepare(int64_t, int64_t, const int32_t*, const int32_t*, int32_t*, int32_t*, int32_t*,
                  cudaStream_t, bool padded = false);
int graph_validate(int64_t, int64_t, const int32_t*, const int32_t*, int32_t*, cudaStream_t);

namespace {

template <class Key>
void pack_sorted(const std::vector<Record>& rec, int n_keys, Key key, std::vector<PackedRecord>& out,
                 std::vector<int32_t>& start, int which, std::vector<double>& val64) {
    std::vector<Record> r = rec;
    std::stable_sort(r.begin(), r.end(), [&](const Record& a, const Record& b) { return key(a) < key(b); });
    out.clear();
    val64.clear();
    for (const Record& x : r) val64.push_back(x.val);
    start.assign(n_keys + 1, 0);
    for (const Record& x : r) {
        PackedRecord p{};
        if (which == 0) { p.a = (uint8_t)x.i1; p.b = (uint8_t)x.i2; }
        if (which == 1) { p.a = (uint8_t)x.i0; p.b = (uint8_t)x.i2; }
        if (which == 2) { p.a = (uint8_t)x.i0; p.b = (uint8_t)x.i1; }
        p.c = (uint8_t)x.i3;
        p.val = (float)x.val;
        out.push_back(p);
        start[key(x) + 1] += 1;
    }
    for (int i = 0; i < n_keys; ++i) start[i + 1] += start[i];
}

}  // namespace

int get_device_tables(const e3j_plan* plan, DeviceTables& out) {
    int device = 0;
    E3J_CUDA_TRY(cudaGetDevice(&device));
    std::lock_guard<std::mutex> lock(plan->mu);
    for (const DeviceTables& t : plan->dev)
        if (t.device == device) { out = t; return E3J_OK; }

    std::vector<PackedRecord> r0, r1, r2;
    std::vector<int32_t> s0, s1, s2, i0_path(plan->D), path_off(plan->P + 1), path_rows(plan->P);
    std::vector<double> v0, v1, v2;
    pack_sorted(plan->rec, plan->D, [](const Record& r) { return r.i0; }, r0, s0, 0, v0);
    pack_sorted(plan->rec, plan->d, [](const Record& r) { return r.i1; }, r1, s1, 1, v1);
    pack_sorted(plan->rec, plan->dp, [](const Record& r) { return r.i2; }, r2, s2, 2, v2);
    for (int k = 0; k < plan->P; ++k) {
        path_off[k] = plan->paths[k].out_off;
        path_rows[k] = 2 * plan->paths[k].L + 1;
        for (int m = 0; m < 2 * plan->paths[k].L + 1; ++m) i0_path[plan->paths[k].out_off + m] = k;
    }
    path_off[plan->P] = plan->D;

    // one allocation, 256-byte aligned sections
    size_t off = 0;
    auto reserve = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    const size_t nb = sizeof(PackedRecord) * plan->rec.size();
    const size_t o_r0 = reserve(nb), o_r1 = reserve(nb), o_r2 = reserve(nb);
    const size_t o_s0 = reserve(4 * s0.size()), o_s1 = reserve(4 * s1.size()), o_s2 = reserve(4 * s2.size());
    const size_t o_ip = reserve(4 * i0_path.size()), o_po = reserve(4 * path_off.size());
    const size_t o_pr = reserve(4 * path_rows.size());
    const size_t nv = sizeof(double) * plan->rec.size();
    const size_t o_v0 = reserve(nv), o_v1 = reserve(nv), o_v2 = reserve(nv);
    const size_t o_st = reserve(256);
    std::vector<char> host(off, 0);
    std::memcpy(host.data() + o_r0, r0.data(), nb);
    std::memcpy(host.data() + o_r1, r1.data(), nb);
    std::memcpy(host.data() + o_r2, r2.data(), nb);
    std::memcpy(host.data() + o_s0, s0.data(), 4 * s0.size());
    std::memcpy(host.data() + o_s1, s1.data(), 4 * s1.size());
    std::memcpy(host.data() + o_s2, s2.data(), 4 * s2.size());
    std::memcpy(host.data() + o_ip, i0_path.data(), 4 * i0_path.size());
    std::memcpy(host.data() + o_po, path_off.data(), 4 * path_off.size());
    std::memcpy(host.data() + o_pr, path_rows.data(), 4 * path_rows.size());
    std::memcpy(host.data() + o_v0, v0.data(), nv);
    std::memcpy(host.data() + o_v1, v1.data(), nv);
    std::memcpy(host.data() + o_v2, v2.data(), nv);

    DeviceTables t;
    t.device = device;
    E3J_CUDA_TRY(cudaMalloc(&t.base, off));
    const cudaError_t err = cudaMemcpy(t.base, host.data(), off, cudaMemcpyHostToDevice);
    if (err != cudaSuccess) { cudaFree(t.base); return cuda_status(err); }
    char* b = (char*)t.base;
    t.by_i0 = (const PackedRecord*)(b + o_r0);
    t.by_i1 = (const PackedRecord*)(b + o_r1);
    t.by_i2 = (const PackedRecord*)(b + o_r2);
    t.i0_start = (const int32_t*)(b + o_s0);
    t.i1_start = (const int32_t*)(b + o_s1);
    t.i2_start = (const int32_t*)(b + o_s2);
    t.i0_path = (const int32_t*)(b + o_ip);
    t.path_out_off = (const int32_t*)(b + o_po);
    t.path_rows = (const int32_t*)(b + o_pr);
    t.val64_i0 = (const double*)(b + o_v0);
    t.val64_i1 = (const double*)(b + o_v1);
    t.val64_i2 = (const double*)(b + o_v2);
    t.status = (int32_t*)(b + o_st);
    plan->dev.push_back(t);
    out = t;
    return E3J_OK;
}

namespace {

inline int grid_for(int64_t n) {
    int64_t g = std::min<int64_t>(std::max<int64_t>(n, 1), (int64_t)sm_count() * 32);
    return (int)g;
}

// Threads per block for a kernel whose blocks work through `items` items block-wide: whole warps, at most 256, and
// as few idle threads in the last pass as the warp granularity allows (128 items: 128 threads, 416: two passes of 224).
inline int block_for(int64_t items) {
    const int64_t passes = (std::max<int64_t>(items, 1) + 255) / 256;
    const int64_t per_pass = (std::max<int64_t>(items, 1) + passes - 1) / passes;
    return (int)std::min<int64_t>(256, std::max<int64_t>(64, (per_pass + 31) / 32 * 32));
}

inline Dims dims_of(const e3j_plan* p) {
    return Dims{p->nq, p->d, p->dp, p->P, p->D, (p->flags & E3J_PLAN_COLLAPSE_OUTPUTS) ? 1 : 0};
}

// workspace layout shared by fwd and bwd: [rowptr | colptr | sender_perm | kernel scratch]
struct WorkspaceLayout {
    size_t rowptr, colptr, perm, scratch, total;
};
WorkspaceLayout layout(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, bool bwd) {
    WorkspaceLayout L{};
    size_t off = 0;
    L.rowptr = off; off = align_up(off + 4 * (size_t)(n_nodes + 1), 256);
    L.colptr = off; if (bwd) off = align_up(off + 4 * (size_t)(n_nodes + 1), 256);
    L.perm = off;   if (bwd) off = align_up(off + 4 * (size_t)std::max<int64_t>(n_edges, 1), 256);
    L.scratch = off;
    const FastKernels* fk = fast_lookup(plan);
    if (fk && bwd && fk->bwd_scratch_bytes) off += fk->bwd_scratch_bytes(n_nodes, n_edges);
    if (fk && !bwd && fk->fwd_scratch_bytes) off += fk->fwd_scratch_bytes(n_nodes, n_edges);
    L.total = align_up(off, 256);
    return L;
}

// dst[i] += src[i]
__global__ void add_into_kernel(int64_t n, float* __restrict__ dst, const float* __restrict__ src, int vec_ok) {
    const int64_t tid = blockIdx.x * (int64_t)blockDim.x + threadIdx.x, stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t n4 = vec_ok ? n / 4 : 0;
    float4* d4 = reinterpret_cast<float4*>(dst);
    const float4* s4 = reinterpret_cast<const float4*>(src);
    for (int64_t i = tid; i < n4; i += stride) {
        float4 a = d4[i];
        const float4 b = s4[i];
        a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
        d4[i] = a;
    }
    for (int64_t i = 4 * n4 + tid; i < n; i += stride) dst[i] += src[i];
}
int add_into(float* dst, const float* src, size_t n, cudaStream_t st) {
    if (n == 0) return E3J_OK;
    const int vec_ok = (((uintptr_t)dst | (uintptr_t)src) & 15u) == 0;
    add_into_kernel<<<sm_count() * 16, 256, 0, st>>>((int64_t)n, dst, src, vec_ok);
    return after_launch();
}

// workspace of the double backward: [forward ws | backward ws | out-sized | x-sized | sh-sized | w-sized]
struct DoubleBwdLayout {
    size_t fwd, bwd, t_out, t_x, t_sh, t_w, total, fwd_bytes, bwd_bytes;
};
DoubleBwdLayout dbl_layout(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges) {
    DoubleBwdLayout L{};
    L.fwd_bytes = layout(plan, n_nodes, n_edges, false).total;
    L.bwd_bytes = layout(plan, n_nodes, n_edges, true).total;
    size_t off = 0;
    L.fwd = off; off = align_up(off + L.fwd_bytes, 256);
    L.bwd = off; off = align_up(off + L.bwd_bytes, 256);
    L.t_out = off; off = align_up(off + 4 * (size_t)n_nodes * plan->D * plan->nq, 256);
    L.t_x = off; off = align_up(off + 4 * (size_t)n_nodes * plan->d * plan->nq, 256);
    L.t_sh = off; off = align_up(off + 4 * (size_t)n_edges * ((plan->dp + 3) / 4 * 4), 256);
    L.t_w = off; off = align_up(off + 4 * (size_t)n_edges * plan->P * plan->nq, 256);
    L.total = off;
    return L;
}

// Channel rows are read and written as 128-bit vectors and by 16-byte bulk copies: every per-channel array
// must start on a 16-byte boundary (NULL = absent is fine).  A misaligned pointer is refused on the host.
bool aligned16(std::initializer_list<const void*> ptrs) {
    for (const void* q : ptrs)
        if ((uintptr_t)q & 15u) return false;
    return true;
}

int check_workspace(const void* ws, size_t have, size_t need) {
    if (need == 0) return E3J_OK;
    if (!ws || ((uintptr_t)ws & 255u) || have < need) return E3J_ERR_WORKSPACE;
    return E3J_OK;
}

}  // namespace
}  // namespace e3j

using namespace e3j;

extern "C" {

int e3j_plan_create(e3j_plan** out, const char* irreps_in, int sh_lmax, const char* irreps_out,
                    int out_lmax, unsigned flags) {
    if (!out || !irreps_in) return E3J_ERR_INVALID_ARG;
    *out = nullptr;
    e3j_plan* plan = new (std::nothrow) e3j_plan();
    if (!plan) return E3J_ERR_INVALID_ARG;
    int st = E3J_ERR_INVALID_ARG;
    try {
        st = build_plan(*plan, irreps_in, sh_lmax, irreps_out, out_lmax, flags);
        if (st == E3J_OK && !(flags & E3J_PLAN_GENERIC_ONLY)) plan->fast_id = fast_find(plan->signature.c_str());
    } catch (...) {
        st = E3J_ERR_INVALID_ARG;
    }
    if (st != E3J_OK) { delete plan; return st; }
    *out = plan;
    return E3J_OK;
}

int e3j_plan_destroy(e3j_plan* plan) {
    if (!plan) return E3J_OK;
    int prev = 0;
    const bool have_dev = cudaGetDevice(&prev) == cudaSuccess;
    for (DeviceTables& t : plan->dev) {
        if (t.base && cudaSetDevice(t.device) == cudaSuccess) cudaFree(t.base);
    }
    if (have_dev && !plan->dev.empty()) cudaSetDevice(prev);
    delete plan;
    return E3J_OK;
}

int e3j_plan_info(const e3j_plan* plan, e3j_plan_info_t* info) {
    if (!plan || !info) return E3J_ERR_INVALID_ARG;
    info->n_channels = plan->nq; info->d_in = plan->d; info->d_sh = plan->dp;
    info->n_paths = plan->P; info->d_out = plan->D; info->nnz = (int)plan->rec.size();
    info->n_pairs = plan->n_pairs; info->specialised = plan->fast_id >= 0 ? 1 : 0;
    return E3J_OK;
}

const char* e3j_plan_signature(const e3j_plan* plan) { return plan ? plan->signature.c_str() : nullptr; }

int e3j_plan_device_status(const e3j_plan* plan, int32_t* status) {
    if (!plan || !status) return E3J_ERR_INVALID_ARG;
    DeviceTables t;
    if (int s = get_device_tables(plan, t)) return s;
    E3J_CUDA_TRY(cudaDeviceSynchronize());
    E3J_CUDA_TRY(cudaMemcpy(status, t.status, sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (*status != 0) E3J_CUDA_TRY(cudaMemset(t.status, 0, sizeof(int32_t)));
    return E3J_OK;
}

int e3j_plan_paths(const e3j_plan* plan, e3j_path_info_t* paths, int capacity) {
    if (!plan || !paths || capacity < plan->P) return E3J_ERR_INVALID_ARG;
    std::copy(plan->paths.begin(), plan->paths.end(), paths);
    return plan->P;
}

int e3j_plan_records(const e3j_plan* plan, int32_t* i0, int32_t* i1, int32_t* i2, int32_t* i3,
                     double* val, int capacity) {
    if (!plan || !i0 || !i1 || !i2 || !i3 || !val) return E3J_ERR_INVALID_ARG;
    const int n = (int)plan->rec.size();
    if (capacity < n) return E3J_ERR_INVALID_ARG;
    for (int r = 0; r < n; ++r) {
        i0[r] = plan->rec[r].i0; i1[r] = plan->rec[r].i1; i2[r] = plan->rec[r].i2;
        i3[r] = plan->rec[r].i3; val[r] = plan->rec[r].val;
    }
    return n;
}

int e3j_graph_prepare(int64_t n_nodes, int64_t n_edges, const int32_t* senders,
                      const int32_t* receivers, int32_t* rowptr, int32_t* sender_perm,
                      int32_t* colptr, void* stream) {
    if (n_nodes < 0 || n_edges < 0 || n_nodes >= (1ll << 31) - 1 || n_edges >= (1ll << 31) - 1)
        return E3J_ERR_INVALID_ARG;
    if (n_edges > 0 && (!senders || !receivers)) return E3J_ERR_INVALID_ARG;
    if ((sender_perm == nullptr) != (colptr == nullptr)) return E3J_ERR_INVALID_ARG;
    return graph_prepare(n_nodes, n_edges, senders, receivers, rowptr, sender_perm, colptr,
                         (cudaStream_t)stream);
}

int e3j_graph_prepare_padded(int64_t n_nodes, int64_t n_edges, const int32_t* senders,
                             const int32_t* receivers, int32_t* rowptr, int32_t* sender_perm,
                             int32_t* colptr, void* stream) {
    if (n_nodes < 0 || n_edges < 0 || n_nodes >= (1ll << 31) - 1 || n_edges >= (1ll << 31) - 1)
        return E3J_ERR_INVALID_ARG;
    if (n_edges > 0 && (!senders || !receivers)) return E3J_ERR_INVALID_ARG;
    if ((sender_perm == nullptr) != (colptr == nullptr)) return E3J_ERR_INVALID_ARG;
    return graph_prepare(n_nodes, n_edges, senders, receivers, rowptr, sender_perm, colptr,
                         (cudaStream_t)stream, true);
}

int e3j_graph_validate(int64_t n_nodes, int64_t n_edges, const int32_t* senders,
                       const int32_t* receivers, int32_t* status, void* stream) {
    if (n_nodes < 0 || n_edges < 0 || !status) return E3J_ERR_INVALID_ARG;
    if (n_edges > 0 && (!senders || !receivers)) return E3J_ERR_INVALID_ARG;
    return graph_validate(n_nodes, n_edges, senders, receivers, status, (cudaStream_t)stream);
}

size_t e3j_conv_fwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges) {
    if (!plan || n_nodes < 0 || n_edges < 0) return 0;
    return layout(plan, n_nodes, n_edges, false).total;
}

size_t e3j_conv_bwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges) {
    if (!plan || n_nodes < 0 || n_edges < 0) return 0;
    return layout(plan, n_nodes, n_edges, true).total;
}

}  // extern "C"

bool e3j::has_fast_forward(const e3j_plan* plan) {
    const FastKernels* fk = fast_lookup(plan);
    return fk && fk->conv_fwd;
}

int e3j::conv_fwd_impl(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x,
                       const float* sh, const float* w, const int32_t* senders,
                       const int32_t* receivers, const int32_t* rowptr, float* out, void* workspace,
                       size_t workspace_bytes, void* stream, bool padded, const float* edge_vec) {
    if (!plan || n_nodes < 0 || n_edges < 0 || n_nodes >= (1ll << 31) - 1 || n_edges >= (1ll << 31) - 1)
        return E3J_ERR_INVALID_ARG;
    if (plan->nq % 4 != 0) return E3J_ERR_UNSUPPORTED;  // the kernels work on groups of four channels
    if (n_nodes == 0) return E3J_OK;
    if (!out || !x) return E3J_ERR_INVALID_ARG;
    if (n_edges > 0 && ((!sh && !edge_vec) || !w || !senders || !receivers)) return E3J_ERR_INVALID_ARG;
    if (edge_vec && !has_fast_forward(plan)) return E3J_ERR_UNSUPPORTED;   // the table-driven kernel reads sh
    if (!aligned16({x, w, out})) return E3J_ERR_INVALID_ARG;
    if (padded && !rowptr) return E3J_ERR_INVALID_ARG;  // rowptr[n_nodes] is where the kernels learn the edge count
    const int32_t* n_real = padded ? rowptr + n_nodes : nullptr;
    cudaStream_t st = (cudaStream_t)stream;
    const WorkspaceLayout L = layout(plan, n_nodes, n_edges, false);
    if (int s = check_workspace(workspace, workspace_bytes, L.total)) return s;
    char* ws = (char*)workspace;

    const FastKernels* fk = fast_lookup(plan);
    if (fk && fk->conv_fwd && n_edges > 0) {
        DeviceTables t;
        if (int s = get_device_tables(plan, t)) return s;
        ConvArgs a{};
        a.n_nodes = n_nodes; a.n_edges = n_edges; a.x = x; a.sh = sh; a.w = w;
        a.senders = senders; a.receivers = receivers; a.rowptr = rowptr; a.out = out;
        a.workspace = ws + L.scratch; a.workspace_bytes = workspace_bytes - L.scratch; a.stream = st;
        a.status = t.status;
        a.n_real = n_real;
        a.vec = edge_vec;
        return fk->conv_fwd(a);
    }
    if (!rowptr) {
        int32_t* rp = (int32_t*)(ws + L.rowptr);
        if (int s = graph_prepare(n_nodes, n_edges, senders, receivers, rp, nullptr, nullptr, st)) return s;
        rowptr = rp;
    }
    DeviceTables t;
    if (int s = get_device_tables(plan, t)) return s;
    generic::conv_fwd_kernel<false><<<grid_for(n_nodes), block_for((int64_t)plan->D * plan->nq / 4), 0, st>>>(t, dims_of(plan), n_nodes, x, sh, w,
                                                                      senders, rowptr, out);
    return after_launch();
}

extern "C" {

int e3j_conv_fwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x,
                 const float* sh, const float* w, const int32_t* senders,
                 const int32_t* receivers, const int32_t* rowptr, float* out, void* workspace,
                 size_t workspace_bytes, void* stream) {
    return conv_fwd_impl(plan, n_nodes, n_edges, x, sh, w, senders, receivers, rowptr, out, workspace,
                         workspace_bytes, stream, false);
}

int e3j_conv_fwd_padded(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges_padded, const float* x,
                        const float* sh, const float* w, const int32_t* senders,
                        const int32_t* receivers, const int32_t* rowptr, float* out, void* workspace,
                        size_t workspace_bytes, void* stream) {
    return conv_fwd_impl(plan, n_nodes, n_edges_padded, x, sh, w, senders, receivers, rowptr, out, workspace,
                         workspace_bytes, stream, true);
}

}  // extern "C"

int e3j::conv_bwd_impl(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x,
                       const float* sh, const float* w, const int32_t* senders,
                       const int32_t* receivers, const int32_t* rowptr, const int32_t* sender_perm,
                       const int32_t* colptr, const float* grad_out, float* grad_x, float* grad_sh,
                       float* grad_w, void* workspace, size_t workspace_bytes, void* stream, bool padded) {
    if (!plan || n_nodes < 0 || n_edges < 0 || n_nodes >= (1ll << 31) - 1 || n_edges >= (1ll << 31) - 1)
        return E3J_ERR_INVALID_ARG;
    if (plan->nq % 4 != 0) return E3J_ERR_UNSUPPORTED;  // the kernels work on groups of four channels
    if (n_nodes == 0) return E3J_OK;
    if (!x || !grad_out) return E3J_ERR_INVALID_ARG;
    if (n_edges > 0 && (!sh || !w || !senders || !receivers)) return E3J_ERR_INVALID_ARG;
    if ((sender_perm == nullptr) != (colptr == nullptr)) return E3J_ERR_INVALID_ARG;
    if (!aligned16({x, w, grad_out, grad_x, grad_w})) return E3J_ERR_INVALID_ARG;
    if (padded && !rowptr) return E3J_ERR_INVALID_ARG;  // rowptr[n_nodes] is where the kernels learn the edge count
    const int32_t* n_real = padded ? rowptr + n_nodes : nullptr;
    cudaStream_t st = (cudaStream_t)stream;
    const WorkspaceLayout L = layout(plan, n_nodes, n_edges, true);
    if (int s = check_workspace(workspace, workspace_bytes, L.total)) return s;
    char* ws = (char*)workspace;
    if (grad_x && !sender_perm) {
        int32_t* cp = (int32_t*)(ws + L.colptr);
        int32_t* pm = (int32_t*)(ws + L.perm);
        if (int s = graph_prepare(n_nodes, n_edges, senders, receivers, nullptr, pm, cp, st, padded)) return s;
        sender_perm = pm; colptr = cp;
    }
    const FastKernels* fk = fast_lookup(plan);
    // the specialised sweep produces all three cotangents at once; those that are not asked for are computed all the
    // same and not stored (grad_sh, grad_w) or not summed (grad_x)
    if (fk && fk->conv_bwd && n_edges > 0 && (grad_x || grad_sh || grad_w)) {
        DeviceTables t;
        if (int s = get_device_tables(plan, t)) return s;
        ConvArgs a{};
        a.status = t.status;
        a.n_nodes = n_nodes; a.n_edges = n_edges; a.x = x; a.sh = sh; a.w = w;
        a.senders = senders; a.receivers = receivers; a.rowptr = rowptr;
        a.sender_perm = sender_perm; a.colptr = colptr; a.grad_out = grad_out;
        a.grad_x = grad_x; a.grad_sh = grad_sh; a.grad_w = grad_w;
        a.workspace = ws + L.scratch; a.workspace_bytes = workspace_bytes - L.scratch; a.stream = st;
        a.n_real = n_real;
        return fk->conv_bwd(a);
    }
    DeviceTables t;
    if (int s = get_device_tables(plan, t)) return s;
    const Dims dm = dims_of(plan);
    if ((grad_w || grad_sh) && n_edges > 0) {
        generic::conv_bwd_edge_kernel<false><<<grid_for(n_edges), block_for((int64_t)dm.P * dm.nq / 4), 0, st>>>(
            t, dm, n_edges, x, sh, w, senders, receivers, grad_out, grad_w, grad_sh, n_real);
        if (int s = after_launch()) return s;
    }
    if (grad_x) {
        generic::conv_bwd_node_kernel<false><<<grid_for(n_nodes), block_for((int64_t)dm.d * dm.nq / 4), 0, st>>>(
            t, dm, n_nodes, sh, w, receivers, sender_perm, colptr, grad_out, grad_x);
        if (int s = after_launch()) return s;
    }
    return E3J_OK;
}

extern "C" {

int e3j_conv_bwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x,
                 const float* sh, const float* w, const int32_t* senders,
                 const int32_t* receivers, const int32_t* rowptr, const int32_t* sender_perm,
                 const int32_t* colptr, const float* grad_out, float* grad_x, float* grad_sh,
                 float* grad_w, void* workspace, size_t workspace_bytes, void* stream) {
    return conv_bwd_impl(plan, n_nodes, n_edges, x, sh, w, senders, receivers, rowptr, sender_perm, colptr,
                         grad_out, grad_x, grad_sh, grad_w, workspace, workspace_bytes, stream, false);
}

int e3j_conv_bwd_padded(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges_padded, const float* x,
                        const float* sh, const float* w, const int32_t* senders,
                        const int32_t* receivers, const int32_t* rowptr, const int32_t* sender_perm,
                        const int32_t* colptr, const float* grad_out, float* grad_x, float* grad_sh,
                        float* grad_w, void* workspace, size_t workspace_bytes, void* stream) {
    return conv_bwd_impl(plan, n_nodes, n_edges_padded, x, sh, w, senders, receivers, rowptr, sender_perm,
                         colptr, grad_out, grad_x, grad_sh, grad_w, workspace, workspace_bytes, stream, true);
}

size_t e3j_conv_bwd_bwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges) {
    if (!plan || n_nodes < 0 || n_edges < 0) return 0;
    return dbl_layout(plan, n_nodes, n_edges).total;
}

int e3j_conv_bwd_bwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x,
                     const float* sh, const float* w, const int32_t* senders,
                     const int32_t* receivers, const int32_t* rowptr, const int32_t* sender_perm,
                     const int32_t* colptr, const float* grad_out, const float* ct_x,
                     const float* ct_sh, const float* ct_w, float* gg_out, float* g_x, float* g_sh,
                     float* g_w, void* workspace, size_t workspace_bytes, void* stream) {
    if (!plan || n_nodes < 0 || n_edges < 0 || n_nodes >= (1ll << 31) - 1 || n_edges >= (1ll << 31) - 1)
        return E3J_ERR_INVALID_ARG;
    if (plan->nq % 4 != 0) return E3J_ERR_UNSUPPORTED;
    if (n_nodes == 0) return E3J_OK;
    if (!x || !grad_out) return E3J_ERR_INVALID_ARG;
    if (n_edges > 0 && (!sh || !w || !senders || !receivers)) return E3J_ERR_INVALID_ARG;
    if (!rowptr || !sender_perm || !colptr) return E3J_ERR_INVALID_ARG;  // six passes: prepare the graph once
    if (!aligned16({x, w, grad_out, ct_x, ct_w, gg_out, g_x, g_w})) return E3J_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const DoubleBwdLayout L = dbl_layout(plan, n_nodes, n_edges);
    if (int s = check_workspace(workspace, workspace_bytes, L.total)) return s;
    char* ws = (char*)workspace;
    float* t_out = (float*)(ws + L.t_out);
    float* t_x = (float*)(ws + L.t_x);
    float* t_sh = (float*)(ws + L.t_sh);
    float* t_w = (float*)(ws + L.t_w);
    const size_t n_out = (size_t)n_nodes * plan->D * plan->nq, n_x = (size_t)n_nodes * plan->d * plan->nq;
    const size_t n_sh = (size_t)n_edges * plan->dp, n_w = (size_t)n_edges * plan->P * plan->nq;

    const FastKernels* fk = fast_lookup(plan);
    // cotangent of grad_out: the forward map with one argument replaced by its cotangent, three times
    // (or the fused sweep of a specialised signature)
    if (gg_out && fk && fk->dbl_out && n_edges > 0 && ct_x && ct_sh && ct_w) {
        DeviceTables t;
        if (int s = get_device_tables(plan, t)) return s;
        const WorkspaceLayout W = layout(plan, n_nodes, n_edges, false);
        ConvArgs a{};
        a.status = t.status;
        a.n_nodes = n_nodes; a.n_edges = n_edges; a.x = x; a.sh = sh; a.w = w;
        a.senders = senders; a.receivers = receivers; a.rowptr = rowptr; a.out = gg_out;
        a.workspace = ws + L.fwd + W.scratch; a.workspace_bytes = L.fwd_bytes - W.scratch; a.stream = st;
        if (int s = fk->dbl_out(a, ct_x, ct_sh, ct_w)) return s;
    } else if (gg_out) {
        bool first = true;
        const float* xs[3] = {ct_x, x, x};
        const float* ys[3] = {sh, ct_sh, sh};
        const float* wsrc[3] = {w, w, ct_w};
        const float* cts[3] = {ct_x, ct_sh, ct_w};
        for (int term = 0; term < 3; ++term) {
            if (!cts[term]) continue;
            float* dst = first ? gg_out : t_out;
            if (int s = conv_fwd_impl(plan, n_nodes, n_edges, xs[term], ys[term], wsrc[term], senders, receivers,
                                      rowptr, dst, ws + L.fwd, L.fwd_bytes, stream, false)) return s;
            if (!first)
                if (int s = add_into(gg_out, t_out, n_out, st)) return s;
            first = false;
        }
        if (first) E3J_CUDA_TRY(cudaMemsetAsync(gg_out, 0, 4 * n_out, st));
    }
    // cotangents of x, sh, w: the backward map with one primal replaced by its cotangent; each pass yields the
    // two cotangents that are not the replaced argument's own (all three are computed so that the specialised
    // sweep can be used; the third goes to scratch)
    if (fk && fk->dbl_edges && n_edges > 0 && ct_x && ct_sh && ct_w && g_x && g_sh && g_w) {
        // one fused sweep instead of the three backward passes below
        DeviceTables t;
        if (int s = get_device_tables(plan, t)) return s;
        const WorkspaceLayout W = layout(plan, n_nodes, n_edges, true);
        ConvArgs a{};
        a.status = t.status;
        a.n_nodes = n_nodes; a.n_edges = n_edges; a.x = x; a.sh = sh; a.w = w;
        a.senders = senders; a.receivers = receivers; a.rowptr = rowptr;
        a.sender_perm = sender_perm; a.colptr = colptr; a.grad_out = grad_out;
        a.grad_x = g_x; a.grad_sh = g_sh; a.grad_w = g_w;
        a.workspace = ws + L.bwd + W.scratch; a.workspace_bytes = L.bwd_bytes - W.scratch; a.stream = st;
        return fk->dbl_edges(a, ct_x, ct_sh, ct_w);
    }
    bool have_x = false, have_sh = false, have_w = false;
    auto put = [&](float* dst, float* tmp, bool& have, size_t n) -> int {
        // result of this pass is in `have ? tmp : dst`; fold it into dst
        if (!dst) return E3J_OK;
        if (have) return add_into(dst, tmp, n, st);
        have = true;
        return E3J_OK;
    };
    if ((g_sh || g_w) && ct_x) {   // x <- ct_x: contributes to sh and w
        float* o_sh = g_sh ? g_sh : t_sh;
        float* o_w = g_w ? g_w : t_w;
        if (int s = conv_bwd_impl(plan, n_nodes, n_edges, ct_x, sh, w, senders, receivers, rowptr, sender_perm, colptr,
                                  grad_out, t_x, o_sh, o_w, ws + L.bwd, L.bwd_bytes, stream, false)) return s;
        have_sh = g_sh != nullptr; have_w = g_w != nullptr;
    }
    if ((g_x || g_w) && ct_sh) {   // sh <- ct_sh: contributes to x and w
        float* o_x = g_x ? g_x : t_x;
        float* o_w = (g_w && !have_w) ? g_w : t_w;
        if (int s = conv_bwd_impl(plan, n_nodes, n_edges, x, ct_sh, w, senders, receivers, rowptr, sender_perm, colptr,
                                  grad_out, o_x, t_sh, o_w, ws + L.bwd, L.bwd_bytes, stream, false)) return s;
        have_x = g_x != nullptr;
        if (int s = put(g_w, t_w, have_w, n_w)) return s;
    }
    if ((g_x || g_sh) && ct_w) {   // w <- ct_w: contributes to x and sh
        float* o_x = (g_x && !have_x) ? g_x : t_x;
        float* o_sh = (g_sh && !have_sh) ? g_sh : t_sh;
        if (int s = conv_bwd_impl(plan, n_nodes, n_edges, x, sh, ct_w, senders, receivers, rowptr, sender_perm, colptr,
                                  grad_out, o_x, o_sh, t_w, ws + L.bwd, L.bwd_bytes, stream, false)) return s;
        if (int s = put(g_x, t_x, have_x, n_x)) return s;
        if (int s = put(g_sh, t_sh, have_sh, n_sh)) return s;
    }
    if (g_x && !have_x) E3J_CUDA_TRY(cudaMemsetAsync(g_x, 0, 4 * n_x, st));
    if (g_sh && !have_sh) E3J_CUDA_TRY(cudaMemsetAsync(g_sh, 0, 4 * n_sh, st));
    if (g_w && !have_w) E3J_CUDA_TRY(cudaMemsetAsync(g_w, 0, 4 * n_w, st));
    return E3J_OK;
}

int e3j_tp_fwd(const e3j_plan* plan, int64_t rows, const float* x1, const float* x2,
               const float* w, float* out, void* stream) {
    if (!plan || rows < 0) return E3J_ERR_INVALID_ARG;
    if (plan->nq % 4 != 0) return E3J_ERR_UNSUPPORTED;  // the kernels work on groups of four channels
    if (rows == 0) return E3J_OK;
    if (!x1 || !x2 || !w || !out) return E3J_ERR_INVALID_ARG;
    if (!aligned16({x1, w, out})) return E3J_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const FastKernels* fk = fast_lookup(plan);
    if (fk && fk->tp_fwd) return fk->tp_fwd(rows, x1, x2, w, out, st);
    DeviceTables t;
    if (int s = get_device_tables(plan, t)) return s;
    generic::conv_fwd_kernel<true><<<grid_for(rows), block_for((int64_t)plan->D * plan->nq / 4), 0, st>>>(t, dims_of(plan), rows, x1, x2, w, nullptr,
                                                                  nullptr, out);
    return after_launch();
}

int e3j_tp_bwd(const e3j_plan* plan, int64_t rows, const float* x1, const float* x2,
               const float* w, const float* grad_out, float* grad_x1, float* grad_x2,
               float* grad_w, void* stream) {
    if (!plan || rows < 0) return E3J_ERR_INVALID_ARG;
    if (plan->nq % 4 != 0) return E3J_ERR_UNSUPPORTED;  // the kernels work on groups of four channels
    if (rows == 0) return E3J_OK;
    if (!x1 || !x2 || !w || !grad_out) return E3J_ERR_INVALID_ARG;
    if (!aligned16({x1, w, grad_out, grad_x1, grad_w})) return E3J_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const FastKernels* fk = fast_lookup(plan);
    if (fk && fk->tp_bwd && grad_x1 && grad_x2 && grad_w)
        return fk->tp_bwd(rows, x1, x2, w, grad_out, grad_x1, grad_x2, grad_w, st);
    DeviceTables t;
    if (int s = get_device_tables(plan, t)) return s;
    const Dims dm = dims_of(plan);
    if (grad_w || grad_x2) {
        generic::conv_bwd_edge_kernel<true><<<grid_for(rows), block_for((int64_t)dm.P * dm.nq / 4), 0, st>>>(t, dm, rows, x1, x2, w, nullptr,
                                                                           nullptr, grad_out, grad_w, grad_x2, nullptr);
        if (int s = after_launch()) return s;
    }
    if (grad_x1) {
        generic::conv_bwd_node_kernel<true><<<grid_for(rows), block_for((int64_t)dm.d * dm.nq / 4), 0, st>>>(t, dm, rows, x2, w, nullptr, nullptr,
                                                                           nullptr, grad_out, grad_x1);
        if (int s = after_launch()) return s;
    }
    return E3J_OK;
}

int e3j_selftest_bounded_wait(const e3j_plan* plan, uint32_t spin_limit, int32_t* returned, int32_t* abort_flag) {
    if (!plan || !returned || !abort_flag || spin_limit == 0 || spin_limit > (1u << 20)) return E3J_ERR_INVALID_ARG;
    DeviceTables t;
    if (int s = get_device_tables(plan, t)) return s;
    // two result words behind the status word, in the plan's own device allocation (its last 256-byte section)
    int32_t* result = t.status + 8;
    fast::bounded_wait_selftest_kernel<<<1, 32>>>(spin_limit, t.status, result);
    if (int s = after_launch()) return s;
    E3J_CUDA_TRY(cudaDeviceSynchronize());
    int32_t host[2] = {0, 0};
    E3J_CUDA_TRY(cudaMemcpy(host, result, sizeof(host), cudaMemcpyDeviceToHost));
    *returned = host[0]; *abort_flag = host[1];
    return E3J_OK;
}

const char* e3j_status_string(int status) {
    switch (status) {
        case E3J_OK: return "ok";
        case E3J_ERR_INVALID_ARG: return "invalid argument";
        case E3J_ERR_BAD_IRREPS: return "irreps descriptor does not parse";
        case E3J_ERR_MUL_NOT_UNIFORM: return "input irreps must share one multiplicity";
        case E3J_ERR_UNSUPPORTED: return "unsupported plan (a dimension exceeds 255, l > 8, no path couples, or channels not a multiple of 4)";
        case E3J_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case E3J_ERR_CUDA: return "CUDA runtime error";
        case E3J_ERR_GRAPH: return "graph invalid (receivers not sorted or index out of range)";
        default: return "unknown status";
    }
}

int e3j_last_cuda_error(void) { return g_last_cuda_error; }
int64_t e3j_launch_count(void) { return g_launch_count.load(std::memory_order_relaxed); }

}  // extern "C"
