/* e3j.h -- C ABI of the B200 (sm_100a) fused equivariant message-passing convolution.
 *
 * The operation (paper: appendix "Tensor Product and Message Passing Convolution
 * kernels", section "Mathematical Details"):
 *
 *   forward  (message-passing-convolution equation)
 *     out[b,i0,q] = sum_{edges e with receiver b} w[e,i3(i0),q]
 *                   * sum_{i1,i2} C[i0,i1,i2] * x[sender(e),i1,q] * sh[e,i2]
 *   backward (message-passing-backward equation, ds per irreducible block)
 *     grad_x[a,i1,q] = sum_{edges e with sender a} sum C * sh[e,i2] * w[e,k,q] * grad_out[b,i0,q]
 *     grad_sh[e,i2]  = sum_q sum C * x[a,i1,q] * w[e,k,q] * grad_out[b,i0,q]
 *     grad_w[e,k,q]  = sum_{i0 in block k} grad_out[b,i0,q] * sum C * x[a,i1,q] * sh[e,i2]
 *
 * C is the real Clebsch-Gordan coupling tensor of every allowed path
 * (l1,p1) x (l2,(-1)^l2) -> (L, p1*(-1)^l2), |l1-l2| <= L <= l1+l2, kept as a
 * sparse list of records (i0,i1,i2,i3,value) sorted by output coordinate i0
 * (paper: "CUDA kernels", sparse COO records).  One output block and one weight
 * block per path (output multiplicities are not collapsed).
 *
 * Conventions
 *   - Layout is the paper's trailing-channel layout: [batch, feature coordinate,
 *     channel], channel fastest.  (The multiplicity-major layout of e3nn is not
 *     accepted; transpose first.)
 *   - Components of a degree-l block are ordered m = -l..l.
 *   - Coefficients: unitary real CG (sum over (m1,m2) of C^2 = 1 per output
 *     component), real basis Y_{l,m>0} = sqrt2 (-1)^m Re Y_l^m,
 *     Y_{l,m<0} = sqrt2 (-1)^m Im Y_l^{|m|}; each path's sign is chosen so that
 *     its first non-zero entry in (M,m1,m2) order is positive
 *     (so 1 x 1 -> 0 is +dot/sqrt(3), l x 0 -> l is +identity).
 *   - Paths are ordered by the position of their output irrep in `irreps_out`
 *     (default 0e,0o,1o,1e,2e,2o,3o,3e,...), ties by (input irrep index, l2).
 *     Output block k and weight block k belong to path k.
 *   - All tensors are float32, all graph indices int32, all pointers DEVICE
 *     pointers unless stated otherwise.  The caller owns every tensor and every
 *     workspace; a plan owns only its coefficient tables.
 *   - Every compute call enqueues work on `stream` (a cudaStream_t passed as
 *     void*) and returns without synchronising.  Outputs are fully overwritten.
 *   - Results are bit-identical from run to run on the same device: no
 *     floating-point atomics are used anywhere.
 *   - There is no CPU fallback.  Without a usable CUDA device every compute call
 *     returns E3J_ERR_CUDA.
 *
 * Alignment: arrays with a channel axis (x, w, out, grad_out and their gradients
 * and cotangents) are read and written as 128-bit vectors and by 16-byte bulk
 * copies, so they must start on a 16-byte boundary; a compute call given a
 * misaligned one returns E3J_ERR_INVALID_ARG without launching anything.  The
 * harmonics (sh) and the index arrays need only their natural 4-byte alignment.
 *
 * Errors: every function returns an int status (0 = E3J_OK, negative = error);
 * nothing throws across this boundary.  e3j_status_string() names a status,
 * e3j_last_cuda_error() returns the cudaError_t behind the last E3J_ERR_CUDA
 * on the calling thread.
 */
#ifndef E3J_H_
#define E3J_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    E3J_OK = 0,
    E3J_ERR_INVALID_ARG = -1,   /* NULL pointer, negative size, capacity too small; compute
                                   calls: a per-channel array not 16-byte aligned            */
    E3J_ERR_BAD_IRREPS = -2,    /* descriptor string does not parse                         */
    E3J_ERR_MUL_NOT_UNIFORM = -3, /* input irreps must share one multiplicity (= N_q)       */
    E3J_ERR_UNSUPPORTED = -4,   /* a dimension exceeds 255, l > 8, nothing couples; compute
                                   calls: channel count N_q not a multiple of 4              */
    E3J_ERR_WORKSPACE = -5,     /* workspace NULL, misaligned (256 B) or too small            */
    E3J_ERR_CUDA = -6,          /* a CUDA runtime call failed; see e3j_last_cuda_error()      */
    E3J_ERR_GRAPH = -7          /* written by e3j_graph_validate into its device status word */
};

/* plan flags */
#define E3J_PLAN_GENERIC_ONLY 1u /* never pick a signature-specialised kernel */
/* Collapsed output multiplicities (paper: the coefficient set of the comparison with the SO(2) convolution, in
 * which the copies of one irreducible output space that different paths produce are added together): all paths
 * that land on the same (L, p) share one output block, out[b, block(L,p) + M, q] = sum over those paths of
 * w[e, path, q] * (...), so D = sum over distinct (L, p) of (2L + 1) while the weights stay one block per
 * path.  out_off of e3j_path_info_t is then the same for the paths of a block.  Such plans use generated
 * kernels where a collapsed signature has been generated (the water-box signature), the table-driven kernels
 * otherwise. */
#define E3J_PLAN_COLLAPSE_OUTPUTS 2u
/* e3j_conv_radial_fwd / e3j_conv_radial_vec_fwd take the two-step form (edge weights written to the workspace by the
 * tensor-core product, then the plain forward) even where the plan has the kernel that forms them itself: faster
 * where the [n_edges, P, N_q] array fits in memory (bench workload: 0.49 against 0.71 ms), at the price of that
 * array in the workspace. */
#define E3J_PLAN_RADIAL_MATERIALISE 4u

typedef struct e3j_plan e3j_plan; /* opaque; immutable after creation; usable from several streams */

typedef struct {
    int n_channels; /* N_q : uniform multiplicity of the input irreps                  */
    int d_in;       /* d   : input feature coordinates, sum (2 l1 + 1)                 */
    int d_sh;       /* d'  : (sh_lmax + 1)^2                                           */
    int n_paths;    /* P   : paths = output blocks = weight blocks                     */
    int d_out;      /* D   : output coordinates, sum over paths (2L + 1)               */
    int nnz;        /* non-zero coefficient records                                    */
    int n_pairs;    /* distinct (i0,i1) pairs with a non-zero coefficient              */
    int specialised;/* 1 if signature-specialised kernels exist and are enabled        */
} e3j_plan_info_t;

typedef struct {
    int in_index;   /* which input irrep                */
    int l1, p1;     /* its degree and parity (+1 / -1)  */
    int l2;         /* harmonic degree                  */
    int L, p;       /* output degree and parity         */
    int x_off;      /* first i1 coordinate              */
    int y_off;      /* first i2 coordinate (= l2^2)     */
    int out_off;    /* first i0 coordinate              */
} e3j_path_info_t;

/* Plan builder (host only; paper: "Reconstruction of Clebsch Gordan coefficients",
 * ladder-operator construction, and "CUDA kernels", sparse records and index packing).
 *   irreps_in   e.g. "128x0e+128x1o"; one multiplicity for all irreps (= N_q)
 *   sh_lmax     harmonics are 1x0e + 1x1o + ... + 1x(sh_lmax)
 *   irreps_out  filter and block order, e.g. "0e+1o+1e+2e+2o"; NULL = every
 *               reachable (L,p) with L <= out_lmax in the default order
 *   out_lmax    used only when irreps_out is NULL; negative = no limit
 * Creates host tables only; device copies are made on first use on each device.
 * The plan must be released with e3j_plan_destroy. */
int e3j_plan_create(e3j_plan** out, const char* irreps_in, int sh_lmax, const char* irreps_out,
                    int out_lmax, unsigned flags);
int e3j_plan_destroy(e3j_plan* plan);
int e3j_plan_info(const e3j_plan* plan, e3j_plan_info_t* info);
/* Canonical text of the plan's signature (multiplicity | input irreps | sh_lmax | paths);
 * specialised kernels are selected by it.  The string is owned by the plan. */
const char* e3j_plan_signature(const e3j_plan* plan);
/* Reads (and clears) the plan's sticky device status word on the current device into the HOST
 * word *status: 0 = fine, 1 = a bounded wait inside a specialised kernel gave up (the kernel
 * then returned early and its outputs are invalid).  Synchronises the device. */
int e3j_plan_device_status(const e3j_plan* plan, int32_t* status);
/* Copies up to `capacity` path descriptors (host memory); returns P or an error. */
int e3j_plan_paths(const e3j_plan* plan, e3j_path_info_t* paths, int capacity);
/* Copies the coefficient records, sorted by (i0, path, i1, i2), into HOST arrays of
 * `capacity` entries each (val in float64 as built, before rounding to float32);
 * returns nnz or an error.  For uncollapsed plans every output row belongs to one path and
 * the order equals (i0, i1, i2). */
int e3j_plan_records(const e3j_plan* plan, int32_t* i0, int32_t* i1, int32_t* i2, int32_t* i3,
                     double* val, int capacity);

/* Graph preparation (paper: the forward algorithm takes receiver CSR pointers as
 * data; the backward is "message passing on the transposed graph").  Integer work
 * only, all on the device:
 *   rowptr[n_nodes+1]   rowptr[b] = first edge with receiver >= b
 *   sender_perm[n_edges] edge ids sorted by (sender, edge id)
 *   colptr[n_nodes+1]   sender_perm[colptr[a] .. colptr[a+1]) are the edges sent by a
 * receivers must be non-decreasing.  Any output pointer may be NULL (skipped);
 * sender_perm and colptr are produced together. */
int e3j_graph_prepare(int64_t n_nodes, int64_t n_edges, const int32_t* senders,
                      const int32_t* receivers, int32_t* rowptr, int32_t* sender_perm,
                      int32_t* colptr, void* stream);
/* Writes 0 (fine) or E3J_ERR_GRAPH (receivers decrease somewhere, or an index is
 * outside [0, n_nodes)) into the DEVICE word *status; read it after synchronising. */
int e3j_graph_validate(int64_t n_nodes, int64_t n_edges, const int32_t* senders,
                       const int32_t* receivers, int32_t* status, void* stream);

/* Convolution forward.  Shapes: x [n_nodes,d,N_q], sh [n_edges,d'], w [n_edges,P,N_q],
 * senders/receivers [n_edges] (receivers non-decreasing), rowptr [n_nodes+1] or NULL
 * (then it is derived into the workspace), out [n_nodes,D,N_q].  Receivers without
 * edges get a row of zeros.  workspace: 256-byte aligned, at least
 * e3j_conv_fwd_workspace_bytes(); its contents need not be preserved between calls,
 * and two calls that overlap on the GPU must not share it. */
size_t e3j_conv_fwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges);
int e3j_conv_fwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x,
                 const float* sh, const float* w, const int32_t* senders,
                 const int32_t* receivers, const int32_t* rowptr, float* out, void* workspace,
                 size_t workspace_bytes, void* stream);

/* Forward convolution without any device allocation or workspace (no counterpart in the paper;
 * added for hosts that cannot allocate).  Some users of this library run where device memory
 * cannot be obtained at call time: a molecular-dynamics engine or an inference server that
 * reserves all of its device memory at start-up and forbids cudaMalloc inside the time-step /
 * request loop, or a plug-in that is handed tensors but has no allocator to make a workspace
 * from.  For them the scratch of the specialised forward kernel lives in a 24 MiB file-scope
 * __device__ array inside the library (every GPU that loads the library holds it until the process
 * exits); the caller passes inputs and the output only.  This function and everything it calls
 * perform no cudaMalloc / cudaFree and no allocating library call.
 *   - Works only for plans with specialised kernels (e3j_plan_info().specialised == 1); other
 *     plans return E3J_ERR_UNSUPPORTED.  A plan whose scratch need on the current device (it
 *     depends on D * N_q and the SM count, not on the graph) exceeds 24 MiB returns
 *     E3J_ERR_WORKSPACE.
 *   - The first call on each device looks the array's address up (cudaGetSymbolAddress, with that
 *     device current) and caches it; make that first call before any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents.
 *     Nothing in it has to be zero at entry (the kernel writes every word before reading it), but
 *     two calls that overlap on the GPU (different streams) race on it: serialise them.
 *   - Results are the same as e3j_conv_fwd's.  A bounded wait that gives up inside the kernel is not
 *     reported through e3j_plan_device_status (that word lives in allocated memory) but through a
 *     status word that is static like the scratch: e3j_noalloc_status reads it into the HOST word
 *     *status and clears it (0 = fine; synchronises the device; allocates nothing).
 * Arguments as for e3j_conv_fwd (receivers non-decreasing; rowptr is not needed). */
int e3j_conv_fwd_noalloc(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x,
                         const float* sh, const float* w, const int32_t* senders,
                         const int32_t* receivers, float* out, void* stream);
int e3j_noalloc_status(int32_t* status);

/* Convolution backward.  grad_out [n_nodes,D,N_q]; grad_x [n_nodes,d,N_q],
 * grad_sh [n_edges,d'], grad_w [n_edges,P,N_q]; any of the three may be NULL (not
 * returned; plans with signature-specialised kernels keep their one sweep and skip the
 * stores of grad_sh / grad_w and the sender sum of grad_x).  rowptr, sender_perm, colptr as produced by e3j_graph_prepare, or NULL
 * (then derived into the workspace on every call).  A node that sends nothing gets
 * a zero grad_x row. */
size_t e3j_conv_bwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges);
int e3j_conv_bwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x,
                 const float* sh, const float* w, const int32_t* senders,
                 const int32_t* receivers, const int32_t* rowptr, const int32_t* sender_perm,
                 const int32_t* colptr, const float* grad_out, float* grad_x, float* grad_sh,
                 float* grad_w, void* workspace, size_t workspace_bytes, void* stream);

/* Padded edge lists (paper: the neighbour list of the molecular-dynamics runs is kept
 * at a fixed padded size and padding edges are flagged; the paper does not give the
 * mechanism, the convention here is): an edge whose receiver id is >= n_nodes is
 * padding.  With receivers non-decreasing the padding edges are the last ones, and the
 * number of real edges is rowptr[n_nodes], which the kernels read on the device - the
 * host never needs it, so a buffer of n_edges_padded entries can be reused while the
 * real count changes.  Nothing of a padding edge is read (its sender, harmonics and
 * weights may hold anything); out and grad_x are those of the real edges; the grad_sh
 * and grad_w rows of padding edges are set to zero.
 * e3j_graph_prepare_padded: as e3j_graph_prepare; sender_perm receives rowptr[n_nodes]
 * entries (the rest is not written), colptr[n_nodes] equals that count.
 * e3j_conv_fwd_padded / e3j_conv_bwd_padded: as e3j_conv_fwd / e3j_conv_bwd with
 * n_edges_padded the length of the edge arrays; rowptr is required (E3J_ERR_INVALID_ARG
 * if NULL) and must come from e3j_graph_prepare_padded (or hold the same values);
 * sender_perm / colptr as produced by it, or NULL (derived into the workspace).
 * Workspace sizes: the e3j_conv_*_workspace_bytes functions with n_edges_padded. */
int e3j_graph_prepare_padded(int64_t n_nodes, int64_t n_edges_padded, const int32_t* senders,
                             const int32_t* receivers, int32_t* rowptr, int32_t* sender_perm,
                             int32_t* colptr, void* stream);
int e3j_conv_fwd_padded(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges_padded, const float* x,
                        const float* sh, const float* w, const int32_t* senders,
                        const int32_t* receivers, const int32_t* rowptr, float* out, void* workspace,
                        size_t workspace_bytes, void* stream);
int e3j_conv_bwd_padded(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges_padded, const float* x,
                        const float* sh, const float* w, const int32_t* senders,
                        const int32_t* receivers, const int32_t* rowptr, const int32_t* sender_perm,
                        const int32_t* colptr, const float* grad_out, float* grad_x, float* grad_sh,
                        float* grad_w, void* workspace, size_t workspace_bytes, void* stream);

/* Double backward (paper: "Differentiation", the double-backward rule needed when the loss contains
 * forces, i.e. gradients of the first backward).  The backward maps (x, sh, w, grad_out) to
 * (grad_x, grad_sh, grad_w).  Given cotangents ct_x, ct_sh, ct_w of those three results (shapes of
 * x, sh, w; any may be NULL = zero) this call returns the cotangents of the backward's four inputs:
 *   gg_out = F(ct_x, sh, w) + F(x, ct_sh, w) + F(x, sh, ct_w)            [n_nodes,D,N_q]   (F = forward map)
 *   g_x    = grad_x of the backward taken at (sh <- ct_sh)  +  at (w <- ct_w)              [n_nodes,d,N_q]
 *   g_sh   = grad_sh at (x <- ct_x)  +  at (w <- ct_w)                                      [n_edges,d']
 *   g_w    = grad_w at (x <- ct_x)   +  at (sh <- ct_sh)                                    [n_edges,P,N_q]
 * all with the same grad_out; any output may be NULL.  In general this is the composition the paper describes
 * (three forward and three backward passes of this library plus the sums).  For signatures with generated
 * double-backward kernels, when all three cotangents are given, it is the fused form the paper leaves as future
 * work: one forward-shaped sweep for gg_out (two terms per coefficient pair) and, if g_x, g_sh and g_w are all
 * wanted, one edge sweep for them (each reads x, sh, w and their cotangents once).  The results of the two forms
 * differ by rounding only.  rowptr, sender_perm and colptr are required (e3j_graph_prepare); the
 * workspace (e3j_conv_bwd_bwd_workspace_bytes) also holds one scratch tensor of each output's size. */
size_t e3j_conv_bwd_bwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges);
int e3j_conv_bwd_bwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x,
                     const float* sh, const float* w, const int32_t* senders,
                     const int32_t* receivers, const int32_t* rowptr, const int32_t* sender_perm,
                     const int32_t* colptr, const float* grad_out, const float* ct_x,
                     const float* ct_sh, const float* ct_w, float* gg_out, float* g_x, float* g_sh,
                     float* g_w, void* workspace, size_t workspace_bytes, void* stream);

/* Edge scalars from the radial network (paper, "Key operations in scope": the scalars of the message-passing
 * layer come from a radial-basis embedding of the interatomic distance followed by a multi-layer perceptron,
 * and scalar mixings are named as candidates for fusion into the message passing; appendix "Mathematical
 * Details", edge scalars).  The last layer of that perceptron is linear, so the per-edge weights are
 *     w[e, k, q] = sum_j h[e, j] * W[j, k * N_q + q]
 * with h [n_edges, hidden] the edge's last hidden activations and W [hidden, P * N_q] the layer's matrix (no
 * bias).  The calls below take (h, W) in place of w, so the [n_edges, P, N_q] weight array, nine tenths of the
 * convolution's minimal memory traffic, is never an input or an output of the call:
 *     out     = conv_fwd(x, sh, h W)
 *     grad_x, grad_sh as in e3j_conv_bwd;  grad_h = grad_w W^T;  grad_W = h^T grad_w   (grad_w internal)
 * The product runs on the tensor cores with every float32 operand split into two TF32 terms (three tensor-core
 * products per float32 product), which keeps float32-level accuracy: results agree with the float64 definition
 * to the same 1e-5 per irreducible block as the other calls, and are bit-identical from run to run (grad_W is
 * summed over fixed edge ranges in a fixed order).
 *   hidden must be a multiple of 4; h, W, grad_h, grad_W 16-byte aligned; rowptr / sender_perm / colptr as for
 *   e3j_conv_fwd / e3j_conv_bwd; any of grad_x, grad_sh, grad_h, grad_W may be NULL.
 *   Workspace: 256-byte aligned, at least e3j_conv_radial_*_workspace_bytes(); calls that overlap on the GPU
 *   must not share it.
 *   The two gradient products fetch their operands through tensor maps (tiled bulk copies); a driver that has no
 *   encoder for them (cuTensorMapEncodeTiled, CUDA 12) makes the backward return E3J_ERR_UNSUPPORTED.
 * e3j_radial_weights writes the product itself, w_out [n_edges, P, N_q] (for callers that want the weights, and
 * as the unfused baseline in measurements). */
int e3j_radial_weights(const e3j_plan* plan, int64_t n_edges, int hidden, const float* h, const float* W,
                       float* w_out, void* stream);
size_t e3j_conv_radial_fwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden);
int e3j_conv_radial_fwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden, const float* x,
                        const float* sh, const float* h, const float* W, const int32_t* senders,
                        const int32_t* receivers, const int32_t* rowptr, float* out, void* workspace,
                        size_t workspace_bytes, void* stream);
size_t e3j_conv_radial_bwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden);
int e3j_conv_radial_bwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden, const float* x,
                        const float* sh, const float* h, const float* W, const int32_t* senders,
                        const int32_t* receivers, const int32_t* rowptr, const int32_t* sender_perm,
                        const int32_t* colptr, const float* grad_out, float* grad_x, float* grad_sh,
                        float* grad_h, float* grad_W, void* workspace, size_t workspace_bytes, void* stream);

/* Standalone channelwise tensor product with per-row, per-path weights (paper:
 * tensor-product formula followed by the edge-scalar weighting; backward: the
 * tensor-product backward rule, one streaming pass).  Rows are their own receivers:
 *   out[r,i0,q] = w[r,i3(i0),q] * sum C[i0,i1,i2] * x1[r,i1,q] * x2[r,i2]
 * x1 [rows,d,N_q], x2 [rows,d'], w [rows,P,N_q], out/grad_out [rows,D,N_q].
 * Any of grad_x1, grad_x2, grad_w may be NULL. */
int e3j_tp_fwd(const e3j_plan* plan, int64_t rows, const float* x1, const float* x2,
               const float* w, float* out, void* stream);
int e3j_tp_bwd(const e3j_plan* plan, int64_t rows, const float* x1, const float* x2,
               const float* w, const float* grad_out, float* grad_x1, float* grad_x2,
               float* grad_w, void* stream);

/* Harmonics of the edge vectors (paper, "Key Operations in Scope": the harmonic embedding Y(r_ab / |r_ab|) of the edge
 * direction is what the convolution takes as sh).  Component normalisation (the squares of the 2l+1 components of a
 * degree sum to 2l+1, Y_0 = 1), degrees stacked l = 0..lmax, m = -l..l inside a degree (l = 1: sqrt(3) (y, z, x)),
 * lmax <= 3.  Device pointers: edge_vec [n_edges, 3] (r_receiver - r_sender, any length), sh / grad_sh
 * [n_edges, (lmax+1)^2] (16-byte aligned), grad_vec [n_edges, 3]; outputs fully overwritten.  The gradient is that of the direction:
 * orthogonal to the vector and proportional to 1 / |vec|.  A zero vector has no direction: its harmonics are the
 * polynomials' values at the origin and its gradient is zero; callers should not pass one. */
int e3j_harmonics_fwd(int lmax, int64_t n_edges, const float* edge_vec, float* sh, void* stream);
int e3j_harmonics_bwd(int lmax, int64_t n_edges, const float* edge_vec, const float* grad_sh, float* grad_vec,
                      void* stream);

/* The convolution on edge vectors instead of harmonics: out = conv_fwd(x, Y(edge_vec), w), and the backward with the
 * chain rule continued into the vectors (grad_vec [n_edges, 3] in place of grad_sh).  The plan's harmonics must be
 * the full set l = 0..lmax, lmax <= 3 (else E3J_ERR_UNSUPPORTED).  Forward: plans with signature-specialised kernels
 * form the harmonics inside the convolution kernel (no [n_edges, d'] array is read or written); other plans run
 * e3j_harmonics_fwd into the workspace first.  Backward: composed (harmonics into the workspace, e3j_conv_bwd,
 * e3j_harmonics_bwd).  Other arguments, alignment and determinism as for e3j_conv_fwd / e3j_conv_bwd; any of
 * grad_x, grad_vec, grad_w may be NULL.  Workspace: 256-byte aligned, e3j_conv_vec_*_workspace_bytes(). */
size_t e3j_conv_vec_fwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges);
size_t e3j_conv_vec_bwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges);
int e3j_conv_vec_fwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x, const float* edge_vec,
                     const float* w, const int32_t* senders, const int32_t* receivers, const int32_t* rowptr,
                     float* out, void* workspace, size_t workspace_bytes, void* stream);
int e3j_conv_vec_bwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x, const float* edge_vec,
                     const float* w, const int32_t* senders, const int32_t* receivers, const int32_t* rowptr,
                     const int32_t* sender_perm, const int32_t* colptr, const float* grad_out, float* grad_x,
                     float* grad_vec, float* grad_w, void* workspace, size_t workspace_bytes, void* stream);

/* Both at once: the forward convolution from edge vectors and the radial layer, out = conv_fwd(x, Y(edge_vec), h W).
 * Where the plan has the kernel that forms the edge scalars itself (see e3j_conv_radial_fwd) that kernel forms the
 * harmonics too, and the call reads x, edge_vec, h, W and the graph only; otherwise the call is composed
 * (e3j_harmonics_fwd and e3j_radial_weights into the workspace, then e3j_conv_fwd).  Arguments as for
 * e3j_conv_radial_fwd with edge_vec [n_edges, 3] in place of sh. */
size_t e3j_conv_radial_vec_fwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden);
int e3j_conv_radial_vec_fwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden, const float* x,
                            const float* edge_vec, const float* h, const float* W, const int32_t* senders,
                            const int32_t* receivers, const int32_t* rowptr, float* out, void* workspace,
                            size_t workspace_bytes, void* stream);

/* Scheduled backward (no counterpart in the paper; it replaces the atomics of the paper's GPU backward and most of the
 * per-edge share array of e3j_conv_bwd's fixed-order sender sum).  The schedule is a processing order of the edges,
 * built once per neighbour list: inside every CTA's edge range, edges with the same sender and neighbouring receivers
 * follow one another in one consumer warp, which adds their shares of grad_x in registers and writes one row per run;
 * the sender sum then reads 1.6 times fewer rows (water box) in a fixed order.  Results are bit-identical from run to
 * run; they differ from e3j_conv_bwd's in the rounding of grad_x only (another, equally fixed, summation order).
 *   e3j_bwd_schedule_bytes      device bytes a schedule may need (0: the plan has no scheduled kernel)
 *   e3j_bwd_schedule_build      senders / receivers are HOST arrays here (receiver-sorted, as everywhere); the order
 *                               is computed on the host and copied to schedule_dev (256-byte aligned) on the stream;
 *                               E3J_ERR_INVALID_ARG for an unsorted list or an index out of range.  The schedule
 *                               belongs to the plan's signature and to the device's SM count.
 *   e3j_conv_bwd_scheduled      e3j_conv_bwd on a schedule: x, sh, w, grad_out and the three gradients as there (all
 *                               three required), workspace as for e3j_conv_bwd.
 *   e3j_bwd_schedule_build_host host-only form for tests and tools: T = edges per tile, writes the schedule's words
 *                               (layout: csrc/bwd_schedule.hpp) to host memory; -2 with *n_words = need if it does
 *                               not fit. */
size_t e3j_bwd_schedule_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges);
int e3j_bwd_schedule_build(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const int32_t* senders_host,
                           const int32_t* receivers_host, void* schedule_dev, size_t schedule_bytes, void* stream);
int e3j_conv_bwd_scheduled(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const float* x, const float* sh,
                           const float* w, const void* schedule_dev, const float* grad_out, float* grad_x,
                           float* grad_sh, float* grad_w, void* workspace, size_t workspace_bytes, void* stream);
int e3j_bwd_schedule_build_host(int T, int n_ranges, int64_t n_nodes, int64_t n_edges, const int32_t* senders,
                                const int32_t* receivers, int32_t* out_words, size_t capacity_words, size_t* n_words);

/* Backward of the call above, composed: harmonics into the workspace, e3j_conv_radial_bwd with the harmonics' cotangent
 * kept as scratch, e3j_harmonics_bwd.  grad_vec [n_edges, 3] in place of grad_sh; any of grad_x, grad_vec, grad_h,
 * grad_W may be NULL. */
size_t e3j_conv_radial_vec_bwd_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden);
int e3j_conv_radial_vec_bwd(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, int hidden, const float* x,
                            const float* edge_vec, const float* h, const float* W, const int32_t* senders,
                            const int32_t* receivers, const int32_t* rowptr, const int32_t* sender_perm,
                            const int32_t* colptr, const float* grad_out, float* grad_x, float* grad_vec,
                            float* grad_h, float* grad_W, void* workspace, size_t workspace_bytes, void* stream);

/* Float64 convolution (paper, appendix on the benchmark setup: float64 builds of the kernels are shipped beside
 * the float32 ones).  Same operation, layouts, graph arguments and conventions as e3j_conv_fwd / e3j_conv_bwd with
 * every tensor in float64 and the coupling coefficients in float64 as the plan builder computed them.  Table-driven
 * kernels for every plan (there are no signature-specialised float64 kernels): each output element is one thread's
 * sum in a fixed order, bit-identical from run to run.  No alignment requirement beyond 8 bytes.  rowptr /
 * sender_perm / colptr as produced by e3j_graph_prepare, or NULL (then derived into the workspace, 256-byte
 * aligned, e3j_conv_f64_workspace_bytes()); any of grad_x, grad_sh, grad_w may be NULL. */
size_t e3j_conv_f64_workspace_bytes(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges);
int e3j_conv_fwd_f64(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const double* x, const double* sh,
                     const double* w, const int32_t* senders, const int32_t* receivers, const int32_t* rowptr,
                     double* out, void* workspace, size_t workspace_bytes, void* stream);
int e3j_conv_bwd_f64(const e3j_plan* plan, int64_t n_nodes, int64_t n_edges, const double* x, const double* sh,
                     const double* w, const int32_t* senders, const int32_t* receivers, const int32_t* sender_perm,
                     const int32_t* colptr, const double* grad_out, double* grad_x, double* grad_sh, double* grad_w,
                     void* workspace, size_t workspace_bytes, void* stream);

/* Receiver sharding over several GPUs, one process per GPU (paper: the one-line SPMD sharding of its API; the
 * backward as message passing on the transposed graph).  A rank owns the receivers [node_lo, node_hi) and the
 * edges into them, a contiguous slice of the receiver-sorted edge list; every edge-local tensor (sh, w, their
 * gradients) and every output row lives with its receiver and never moves.  What crosses GPUs is node rows only:
 * forward, the x rows of the halo (senders the rank does not own); backward, the grad_x shares for those
 * senders, which their owners add in rank order (bit-reproducible).  The exchange itself is the caller's
 * (torch.distributed / NCCL; paper_2609_35099_b200/sharding.py); remote rows land in local memory before any
 * kernel of this library reads them.
 * e3j_shard_prepare: integer kernels.  In: the slice's global sender / receiver ids.  Out: local ids
 *   (owned node node_lo + i -> i; halo node halo_ids[h] -> (node_hi - node_lo) + h), halo_ids in ascending global
 *   order (capacity n_nodes) and the DEVICE word *n_halo.  The local problem then has (node_hi - node_lo) + n_halo
 *   nodes and runs through e3j_graph_prepare / e3j_conv_fwd / e3j_conv_bwd unchanged.
 * e3j_rows_gather: dst[i, :] = src[ids[i], :].  e3j_rows_add: dst[ids[i], :] += src[i, :]; ids must not repeat
 *   within a call (the ids of one rank's halo do not).  row_len floats, a multiple of 4; 16-byte aligned rows. */
size_t e3j_shard_prepare_workspace_bytes(int64_t n_nodes);
int e3j_shard_prepare(int64_t n_nodes, int64_t n_edges_shard, int32_t node_lo, int32_t node_hi,
                      const int32_t* senders, const int32_t* receivers, int32_t* local_senders,
                      int32_t* local_receivers, int32_t* halo_ids, int32_t* n_halo, void* workspace,
                      size_t workspace_bytes, void* stream);
int e3j_rows_gather(float* dst, const float* src, const int32_t* ids, int64_t n_ids, int64_t row_len, void* stream);
int e3j_rows_add(float* dst, const float* src, const int32_t* ids, int64_t n_ids, int64_t row_len, void* stream);

/* Self-test of the kernels' bounded waits (no counterpart in the paper).  Every wait inside the specialised
 * kernels gives up after a fixed number of polls, records the failure in the plan's device status word and
 * lets the kernel drain instead of hanging the GPU.  This call exercises that path on purpose, without any
 * risk of a hang: one warp waits, for at most spin_limit polls (1 .. 2^20), on a barrier that nothing will
 * complete.  On return *returned is what the wait returned (0 = gave up), *abort_flag the kernel's abort flag
 * (1), both HOST words, and e3j_plan_device_status(plan) reads 1 once and 0 afterwards.  Synchronises. */
int e3j_selftest_bounded_wait(const e3j_plan* plan, uint32_t spin_limit, int32_t* returned, int32_t* abort_flag);

const char* e3j_status_string(int status);
int e3j_last_cuda_error(void);
/* Number of kernel launches this library has enqueued from the calling process. */
int64_t e3j_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* E3J_H_ */
