// Internal: registry of signature-specialised kernels (generated, compiled ahead of time).
#pragma once
#include <cstddef>
#include <cstdint>

#include "common.cuh"

namespace e3j {

// The radial network's last layer and the slot tables of the graph (device pointers).
struct RadialArgs {
    const float* h;            // [n_edges, hidden]
    const float* W;            // [hidden, P * N_q]
    int hidden;
    const int32_t* slotptr;    // [n_nodes + 1] first slot of every receiver; slotptr[n_nodes] = number of slots
    const int32_t* slot_edge;  // [slots] edge of the slot, or -1 (padding to a multiple of 8 per receiver)
    const int32_t* group_recv; // [slots / 8] receiver of every group of 8 slots
    void* scratch;             // boundary rows: as for conv_fwd, sized by radial_fwd_scratch_bytes
    size_t scratch_bytes;
};

struct FastKernels {
    const char* signature;  // plan signature this entry was generated for
    size_t (*fwd_scratch_bytes)(int64_t n_nodes, int64_t n_edges);
    size_t (*bwd_scratch_bytes)(int64_t n_nodes, int64_t n_edges);
    int (*conv_fwd)(const ConvArgs&);
    int (*conv_bwd)(const ConvArgs&);
    int (*tp_fwd)(int64_t rows, const float* x1, const float* x2, const float* w, float* out, cudaStream_t);
    int (*tp_bwd)(int64_t rows, const float* x1, const float* x2, const float* w, const float* g,
                  float* gx1, float* gx2, float* gw, cudaStream_t);
    // fused double backward (null: the caller composes it from conv_fwd and conv_bwd).  Cotangents of
    // (grad_x, grad_sh, grad_w) in, both need the scratch of conv_bwd / conv_fwd respectively:
    // dbl_edges writes the cotangents of x, sh, w into args.grad_x / grad_sh / grad_w,
    // dbl_out the cotangent of grad_out into args.out.
    int (*dbl_edges)(const ConvArgs&, const float* ct_x, const float* ct_sh, const float* ct_w);
    int (*dbl_out)(const ConvArgs&, const float* ct_x, const float* ct_sh, const float* ct_w);
    // forward with the edge scalars formed in the kernel from the radial layer (null: the caller materialises
    // them first); see fast/fast_radial.cuh
    int (*radial_fwd)(const ConvArgs&, const RadialArgs&);
    // backward over a processing order built once per neighbour list (fast/fast_bwd1s.cuh, bwd_schedule.hpp);
    // null: the signature has no scheduled kernel.  sched_T = edges per tile the order must be built for.
    int (*conv_bwd_sched)(const ConvArgs&, const int32_t* schedule);
    int sched_T;
};

// Index of the entry generated for `signature`, or -1.
int fast_find(const char* signature);
// Entry selected at plan creation, or nullptr (generic kernels).
const FastKernels* fast_lookup(const e3j_plan* plan);

}  // namespace e3j
