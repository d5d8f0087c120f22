// Convolution with the edge scalars taken from the radial network's last linear layer: s = h W.
//
// This file holds the tensor-core products around that layer (radial_gemm.cuh), the entry point that
// materialises s, and the entry points that run the convolution on (h, W) instead of w.
#include <algorithm>

#include "common.cuh"
#include "fast/fast_launch.cuh"
#include "fast/fast_radial.cuh"
#include "fast_registry.hpp"
#include "radial_gemm.cuh"

namespace e3j {

int graph_prepare(int64_t, int64_t, const int32_t*, const int32_t*, int32_t*, int32_t*, int32_t*, cudaStream_t,
                  bool padded = false);

namespace radial {

__global__ void layer_sum_kernel(int n_ranges, int64_t n_elems, const float* __restrict__ partial,
                                 float* __restrict__ grad_W) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n_elems; i += stride) {
        float acc = partial[i];
        for (int r = 1; r < n_ranges; ++r) acc += partial[(size_t)r * n_elems + i];   // fixed order
        grad_W[i] = acc;
    }
}

namespace {

template <class Prob>
int launch_gemm(const Prob& prob, dim3 grid, cudaStream_t st, int resident_chunks = 0) {
    using L = GemmSmem<Prob::N>;
    static_assert(L::total <= 227 * 1024, "stage ring does not fit in shared memory");
    static_assert(L::res_total(kMaxResidentChunks) <= 227 * 1024, "resident operand does not fit in shared memory");
    constexpr bool kResident = ProbTraits<Prob>::A_RESIDENT;
    constexpr bool kTma = TmaTraits<Prob>::TMA;
    static_assert(!kTma || L::tma_total <= 227 * 1024, "ring of raw boxes does not fit in shared memory");
    constexpr size_t most = kResident ? L::res_total(kMaxResidentChunks) : kTma ? L::tma_total : L::total;
    static thread_local int attr_dev = -1;
    int dev = 0;
    E3J_CUDA_TRY(cudaGetDevice(&dev));
    if (attr_dev != dev) {
        E3J_CUDA_TRY(cudaFuncSetAttribute(gemm_tf32x3_kernel<Prob>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)most));
        attr_dev = dev;
    }
    const size_t bytes = kResident ? L::res_total(resident_chunks) : most;
    gemm_tf32x3_kernel<Prob><<<grid, gemm_threads<Prob>(), bytes, st>>>(prob);
    return after_launch();
}

// Tensor map of a row-major float32 matrix [rows][cols] with `pitch` floats between rows, fetched in boxes of
// box_cols x box_rows.  False where the matrix does not meet the copy engine's alignment rules (16-byte aligned
// base and rows) or the driver has no encoder.
using EncodeTiled = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiled tensor_map_encoder() {
    static const EncodeTiled fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiled>(p);
    }();
    return fn;
}
bool make_map(CUtensorMap* map, const float* base, int64_t rows, int64_t cols, int64_t pitch, int box_cols, int box_rows,
              bool swizzle128) {
    const EncodeTiled encode = tensor_map_encoder();
    if (!encode || (reinterpret_cast<uintptr_t>(base) & 15) || (pitch & 3) || rows <= 0 || cols <= 0) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)pitch * sizeof(float)};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t elem[2] = {1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, elem,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline int64_t round_up(int64_t v, int64_t m) { return (v + m - 1) / m * m; }

}  // namespace

// number of edge ranges of the layer-gradient product on the current device
int layer_ranges(int C) {
    const int n_cb = (C + 127) / 128;
    return std::max(1, fast::sm_count() / n_cb);
}

int radial_weights(int64_t n_edges, int H, int C, const float* h, const float* W, float* s, int32_t* status,
                   cudaStream_t st) {
    if (n_edges == 0) return E3J_OK;
    const int n_cb = (C + 127) / 128;
    const int n_ranges = std::max(1, fast::sm_count() / n_cb);
    RadialWeights p{};
    p.h = h; p.W = W; p.s = s; p.n_edges = n_edges; p.H = H; p.C = C; p.status = status;
    p.chunk = round_up((n_edges + n_ranges - 1) / n_ranges, 128);
    const int chunks = (H + kChunkK - 1) / kChunkK;
    if (chunks > kMaxResidentChunks) {   // a wide hidden layer: W^T converted per tile like the other operand
        RadialWeightsWide q{};
        static_cast<RadialWeights&>(q) = p;
        return launch_gemm(q, dim3(n_cb, n_ranges), st);
    }
    return launch_gemm(p, dim3(n_cb, n_ranges), st, chunks);
}

int grad_hidden(int64_t n_edges, int H, int C, const float* gs, const float* W, float* gh, int32_t* status,
                cudaStream_t st) {
    if (n_edges == 0) return E3J_OK;
    const int n_cta = fast::sm_count();
    GradHidden p{};
    p.gs = gs; p.W = W; p.gh = gh; p.n_edges = n_edges; p.H = H; p.C = C; p.status = status;
    p.chunk = round_up((n_edges + n_cta - 1) / n_cta, 128);
    p.gc = kGroupChunksTma;
    if (!make_map(&p.map_a, gs, n_edges, C, C, kChunkK, 128, true) || !make_map(&p.map_b, W, H, C, C, kChunkK, 64, true))
        return E3J_ERR_UNSUPPORTED;   // (the entry points have checked the alignment: the driver has no encoder)
    return launch_gemm(p, dim3(n_cta, (H + 63) / 64), st);
}

// partial: [layer_ranges(C)][H][C] floats of scratch
int grad_layer(int64_t n_edges, int H, int C, const float* gs, const float* h, float* partial, float* gW,
               int32_t* status, cudaStream_t st) {
    const int64_t n_elems = (int64_t)H * C;
    if (n_edges == 0) {
        E3J_CUDA_TRY(cudaMemsetAsync(gW, 0, sizeof(float) * (size_t)n_elems, st));
        return E3J_OK;
    }
    const int n_cb = (C + 127) / 128, n_ranges = layer_ranges(C);
    GradLayer p{};
    p.gs = gs; p.h = h; p.partial = partial; p.n_edges = n_edges; p.H = H; p.C = C; p.status = status;
    p.chunk = round_up((n_edges + n_ranges - 1) / n_ranges, kChunkK);
    p.gc = kGroupChunksTma;
    if (!make_map(&p.map_a, gs, n_edges, C, C, 128, kChunkK, false) || !make_map(&p.map_b, h, n_edges, H, H, 64, kChunkK, false))
        return E3J_ERR_UNSUPPORTED;
    if (int s = launch_gemm(p, dim3(n_cb, n_ranges, (H + 63) / 64), st)) return s;
    const int blocks = (int)std::min<int64_t>((n_elems + 255) / 256, 4 * fast::sm_count());
    layer_sum_kernel<<<blocks, 256, 0, st>>>(n_ranges, n_elems, partial, gW);
    return after_launch();
}

namespace {

// Does the plan have a kernel that forms the edge scalars itself, for this hidden width?
const FastKernels* fused_forward(const e3j_plan* plan, int H) {
    if (plan->flags & E3J_PLAN_RADIAL_MATERIALISE) return nullptr;
    const FastKernels* fk = fast_lookup(plan);
    return (fk && fk->radial_fwd && fk->fwd_scratch_bytes && H % 8 == 0 && H <= fast::kMaxHidden) ? fk : nullptr;
}

// workspace of the composed calls: [conv workspace | s | grad_s | layer partials]; of the forward with in-kernel
// edge scalars: [rowptr | slotptr | slot_edge | group_recv | boundary-row scratch]
struct RadialLayout {
    size_t conv, s, gs, partial, total, conv_bytes;
    size_t rowptr, slotptr, slot_edge, group_recv, scratch, scratch_bytes;
    bool fused;
};
RadialLayout radial_layout(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int H, bool bwd) {
    RadialLayout L{};
    const size_t C = (size_t)plan->P * plan->nq;
    size_t off = 0;
    const FastKernels* fk = bwd ? nullptr : fused_forward(plan, H);
    if (fk) {
        L.fused = true;
        const size_t cap = (size_t)fast::radial_slot_capacity(n_nodes, n_edges);
        L.rowptr = off; off = align_up(off + 4 * (size_t)(n_nodes + 1), 256);
        L.slotptr = off; off = align_up(off + 4 * (size_t)(n_nodes + 1), 256);
        L.slot_edge = off; off = align_up(off + 4 * cap, 256);
        L.group_recv = off; off = align_up(off + 4 * (cap / fast::kGroup), 256);
        L.scratch_bytes = fk->fwd_scratch_bytes(n_nodes, n_edges);   // sized for more CTAs than there are ranges
        L.scratch = off; off = align_up(off + L.scratch_bytes, 256);
        L.total = off;
        return L;
    }
    L.conv_bytes = bwd ? e3j_conv_bwd_workspace_bytes(plan, n_nodes, n_edges)
                       : e3j_conv_fwd_workspace_bytes(plan, n_nodes, n_edges);
    L.conv = off; off = align_up(off + L.conv_bytes, 256);
    L.s = off; off = align_up(off + 4 * (size_t)std::max<int64_t>(n_edges, 1) * C, 256);
    L.gs = off; if (bwd) off = align_up(off + 4 * (size_t)std::max<int64_t>(n_edges, 1) * C, 256);
    L.partial = off; if (bwd) off = align_up(off + 4 * (size_t)(fast::kMaxSms) * H * C, 256);
    L.total = off;
    return L;
}

bool radial_args_ok(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int H) {
    return plan && n_nodes >= 0 && n_edges >= 0 && n_nodes < (1ll << 31) - 1 && n_edges < (1ll << 31) - 1 && H > 0;
}

}  // namespace
}  // namespace radial
}  // namespace e3j

using namespace e3j;

extern "C" {

int e3j_radial_weights(const e3j_plan* plan, int64_t n_edges, int hidden, const float* h, const float* W,
                       float* w_out, void* stream) {
    if (!radial::radial_args_ok(plan, 0, n_edges, hidden)) return E3J_ERR_INVALID_ARG;
    if (hidden % 4 != 0 || plan->nq % 4 != 0) return E3J_ERR_UNSUPPORTED;
    if (n_edges == 0) return E3J_OK;
    if (!h || !W || !w_out) return E3J_ERR_INVALID_ARG;
    if (((uintptr_t)h | (uintptr_t)W | (uintptr_t)w_out) & 15u) return E3J_ERR_INVALID_ARG;
    DeviceTables t;
    if (int s = get_device_tables(plan, t)) return s;
    return radial::radial_weights(n_edges, hidden, plan->P * plan->nq, h, W, w_out, t.status, (cudaStream_t)stream);
}

size_t e3j_conv_radial_fwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden) {
    if (!radial::radial_args_ok(plan, n_nodes, n_edges, hidden)) return 0;
    return radial::radial_layout(plan, n_nodes, n_edges, hidden, false).total;
}

size_t e3j_conv_radial_bwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden) {
    if (!radial::radial_args_ok(plan, n_nodes, n_edges, hidden)) return 0;
    return radial::radial_layout(plan, n_nodes, n_edges, hidden, true).total;
}

}  // extern "C"

// sh, or edge_vec with sh_scratch (room for [n_edges, d'] floats, used where no kernel forms the harmonics itself)
static int radial_fwd_impl(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden, const float* x,
                           const float* sh, const float* edge_vec, float* sh_scratch, const float* h, const float* W,
                           const int32_t* senders, const int32_t* receivers, const int32_t* rowptr, float* out,
                           void* workspace, size_t workspace_bytes, void* stream) {
    if (!radial::radial_args_ok(plan, n_nodes, n_edges, hidden)) return E3J_ERR_INVALID_ARG;
    if (hidden % 4 != 0 || plan->nq % 4 != 0) return E3J_ERR_UNSUPPORTED;
    if (n_nodes == 0) return E3J_OK;
    if (n_edges > 0 && (!h || !W)) return E3J_ERR_INVALID_ARG;
    if (((uintptr_t)h | (uintptr_t)W) & 15u) return E3J_ERR_INVALID_ARG;
    const radial::RadialLayout L = radial::radial_layout(plan, n_nodes, n_edges, hidden, false);
    if (!workspace || ((uintptr_t)workspace & 255u) || workspace_bytes < L.total) return E3J_ERR_WORKSPACE;
    char* ws = (char*)workspace;
    if (L.fused && n_edges > 0) {
        // edge scalars formed inside the kernel: slot tables of the graph, then one sweep
        if (!x || !out || (!sh && !edge_vec) || !senders || !receivers) return E3J_ERR_INVALID_ARG;
        if (((uintptr_t)x | (uintptr_t)out) & 15u) return E3J_ERR_INVALID_ARG;
        cudaStream_t st = (cudaStream_t)stream;
        if (!rowptr) {
            int32_t* rp = (int32_t*)(ws + L.rowptr);
            if (int rc = graph_prepare(n_nodes, n_edges, senders, receivers, rp, nullptr, nullptr, st)) return rc;
            rowptr = rp;
        }
        int32_t* slotptr = (int32_t*)(ws + L.slotptr);
        int32_t* slot_edge = (int32_t*)(ws + L.slot_edge);
        int32_t* group_recv = (int32_t*)(ws + L.group_recv);
        if (int rc = fast::build_slot_tables(n_nodes, n_edges, rowptr, slotptr, slot_edge, group_recv, st)) return rc;
        DeviceTables t;
        if (int rc = get_device_tables(plan, t)) return rc;
        ConvArgs a{};
        a.n_nodes = n_nodes; a.n_edges = n_edges; a.x = x; a.sh = sh; a.senders = senders; a.receivers = receivers;
        a.rowptr = rowptr; a.out = out; a.stream = st; a.status = t.status;
        a.vec = sh ? nullptr : edge_vec;
        RadialArgs r{};
        r.h = h; r.W = W; r.hidden = hidden; r.slotptr = slotptr; r.slot_edge = slot_edge; r.group_recv = group_recv;
        r.scratch = ws + L.scratch; r.scratch_bytes = L.scratch_bytes;
        return radial::fused_forward(plan, hidden)->radial_fwd(a, r);
    }
    if (L.fused) {   // no edges: every receiver row is empty
        if (!out) return E3J_ERR_INVALID_ARG;
        E3J_CUDA_TRY(cudaMemsetAsync(out, 0, sizeof(float) * (size_t)n_nodes * plan->D * plan->nq, (cudaStream_t)stream));
        return E3J_OK;
    }
    float* s = (float*)(ws + L.s);
    if (n_edges > 0) {
        DeviceTables t;
        if (int st = get_device_tables(plan, t)) return st;
        if (int st = radial::radial_weights(n_edges, hidden, plan->P * plan->nq, h, W, s, t.status, (cudaStream_t)stream))
            return st;
        if (!sh) {   // composed form on edge vectors: the harmonics go through the caller's scratch
            if (!edge_vec || !sh_scratch) return E3J_ERR_INVALID_ARG;
            if (int st = harmonics_fwd(plan_sh_lmax(plan), n_edges, edge_vec, sh_scratch, (cudaStream_t)stream)) return st;
            sh = sh_scratch;
        }
    }
    return conv_fwd_impl(plan, n_nodes, n_edges, x, sh, s, senders, receivers, rowptr, out, ws + L.conv, L.conv_bytes,
                         stream, false);
}

extern "C" {

int e3j_conv_radial_fwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden, const float* x,
                        const float* sh, const float* h, const float* W, const int32_t* senders,
                        const int32_t* receivers, const int32_t* rowptr, float* out, void* workspace,
                        size_t workspace_bytes, void* stream) {
    if (n_edges > 0 && !sh) return E3J_ERR_INVALID_ARG;
    return radial_fwd_impl(plan, n_nodes, n_edges, hidden, x, sh, nullptr, nullptr, h, W, senders, receivers, rowptr, out,
                           workspace, workspace_bytes, stream);
}

size_t e3j_conv_radial_vec_fwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden) {
    if (!radial::radial_args_ok(plan, n_nodes, n_edges, hidden)) return 0;
    return align_up(radial::radial_layout(plan, n_nodes, n_edges, hidden, false).total, 256) +
           align_up(4 * (size_t)std::max<int64_t>(n_edges, 1) * plan->dp, 256);
}

int e3j_conv_radial_vec_fwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden, const float* x,
                            const float* edge_vec, const float* h, const float* W, const int32_t* senders,
                            const int32_t* receivers, const int32_t* rowptr, float* out, void* workspace,
                            size_t workspace_bytes, void* stream) {
    if (!radial::radial_args_ok(plan, n_nodes, n_edges, hidden)) return E3J_ERR_INVALID_ARG;
    if (plan_sh_lmax(plan) < 0) return E3J_ERR_UNSUPPORTED;
    if (n_edges > 0 && !edge_vec) return E3J_ERR_INVALID_ARG;
    const size_t inner = align_up(radial::radial_layout(plan, n_nodes, n_edges, hidden, false).total, 256);
    if (!workspace || ((uintptr_t)workspace & 255u) ||
        workspace_bytes < e3j_conv_radial_vec_fwd_workspace_bytes(plan, n_nodes, n_edges, hidden))
        return E3J_ERR_WORKSPACE;
    return radial_fwd_impl(plan, n_nodes, n_edges, hidden, x, nullptr, edge_vec, (float*)((char*)workspace + inner), h, W,
                           senders, receivers, rowptr, out, workspace, inner, stream);
}

int e3j_conv_radial_bwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden, const float* x,
                        const float* sh, const float* h, const float* W, const int32_t* senders,
                        const int32_t* receivers, const int32_t* rowptr, const int32_t* sender_perm,
                        const int32_t* colptr, const float* grad_out, float* grad_x, float* grad_sh,
                        float* grad_h, float* grad_W, void* workspace, size_t workspace_bytes, void* stream) {
    if (!radial::radial_args_ok(plan, n_nodes, n_edges, hidden)) return E3J_ERR_INVALID_ARG;
    if (hidden % 4 != 0 || plan->nq % 4 != 0) return E3J_ERR_UNSUPPORTED;
    if (n_nodes == 0) return E3J_OK;
    if (!W || (n_edges > 0 && !h)) return E3J_ERR_INVALID_ARG;
    if (((uintptr_t)h | (uintptr_t)W | (uintptr_t)grad_h | (uintptr_t)grad_W) & 15u) return E3J_ERR_INVALID_ARG;
    const radial::RadialLayout L = radial::radial_layout(plan, n_nodes, n_edges, hidden, true);
    if (!workspace || ((uintptr_t)workspace & 255u) || workspace_bytes < L.total) return E3J_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char* ws = (char*)workspace;
    float* s = (float*)(ws + L.s);
    float* gs = (float*)(ws + L.gs);
    const int C = plan->P * plan->nq;
    DeviceTables t;
    if (int rc = get_device_tables(plan, t)) return rc;
    if (int rc = radial::radial_weights(n_edges, hidden, C, h, W, s, t.status, st)) return rc;
    // the convolution's own backward, with the edge-scalar cotangent kept as scratch
    const bool want_gs = grad_h || grad_W;
    if (int rc = conv_bwd_impl(plan, n_nodes, n_edges, x, sh, s, senders, receivers, rowptr, sender_perm, colptr,
                               grad_out, grad_x, grad_sh, want_gs ? gs : nullptr, ws + L.conv, L.conv_bytes, stream,
                               false)) return rc;
    // chain rule through s = h W
    if (grad_h)
        if (int rc = radial::grad_hidden(n_edges, hidden, C, gs, W, grad_h, t.status, st)) return rc;
    if (grad_W)
        if (int rc = radial::grad_layer(n_edges, hidden, C, gs, h, (float*)(ws + L.partial), grad_W, t.status, st)) return rc;
    return E3J_OK;
}

size_t e3j_conv_radial_vec_bwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden) {
    if (!radial::radial_args_ok(plan, n_nodes, n_edges, hidden)) return 0;
    return align_up(radial::radial_layout(plan, n_nodes, n_edges, hidden, true).total, 256) +
           2 * align_up(4 * (size_t)std::max<int64_t>(n_edges, 1) * plan->dp, 256);
}

int e3j_conv_radial_vec_bwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden, const float* x,
                            const float* edge_vec, const float* h, const float* W, const int32_t* senders,
                            const int32_t* receivers, const int32_t* rowptr, const int32_t* sender_perm,
                            const int32_t* colptr, const float* grad_out, float* grad_x, float* grad_vec,
                            float* grad_h, float* grad_W, void* workspace, size_t workspace_bytes, void* stream) {
    if (!radial::radial_args_ok(plan, n_nodes, n_edges, hidden)) return E3J_ERR_INVALID_ARG;
    const int lmax = plan_sh_lmax(plan);
    if (lmax < 0) return E3J_ERR_UNSUPPORTED;
    if (n_edges > 0 && !edge_vec) return E3J_ERR_INVALID_ARG;
    const size_t inner = align_up(radial::radial_layout(plan, n_nodes, n_edges, hidden, true).total, 256);
    const size_t sh_bytes = align_up(4 * (size_t)std::max<int64_t>(n_edges, 1) * plan->dp, 256);
    if (!workspace || ((uintptr_t)workspace & 255u) || workspace_bytes < inner + 2 * sh_bytes) return E3J_ERR_WORKSPACE;
    float* sh = (float*)((char*)workspace + inner);
    float* gsh = (float*)((char*)workspace + inner + sh_bytes);
    cudaStream_t st = (cudaStream_t)stream;
    if (int rc = harmonics_fwd(lmax, n_edges, edge_vec, sh, st)) return rc;
    if (int rc = e3j_conv_radial_bwd(plan, n_nodes, n_edges, hidden, x, sh, h, W, senders, receivers, rowptr, sender_perm,
                                     colptr, grad_out, grad_x, grad_vec ? gsh : nullptr, grad_h, grad_W, workspace, inner,
                                     stream)) return rc;
    if (grad_vec && n_nodes > 0)
        if (int rc = harmonics_bwd(lmax, n_edges, edge_vec, gsh, grad_vec, st)) return rc;
    return E3J_OK;
}

}  // extern "C"
