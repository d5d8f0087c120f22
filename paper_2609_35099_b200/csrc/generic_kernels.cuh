// Table-driven kernels that work for every plan (any irreps, any channel count).
//
// Each output element is owned by exactly one thread and is computed as the
// defining sum in a fixed order, so the results are deterministic without
// atomics.  This is the paper's "transposed record sets" formulation (section
// "Differentiation": for dx the records are sorted by i1, for dy by i2): every
// cotangent is a gather with its own sorted copy of the coefficient records.
// They are the fallback for signatures that have no specialised kernel and the
// on-device cross-check for the specialised ones.
#pragma once
#include "common.cuh"

namespace e3j {
namespace generic {

// IDENT = true: every row is its own sender and receiver (standalone tensor product).
// Threads own groups of four consecutive channels (N_q is a multiple of 4), so every feature, weight and
// cotangent access is a 16-byte load; the coefficient records and harmonics are warp-uniform loads.

__device__ __forceinline__ void f4_fma(float4& acc, const float s, const float4 v) {
    acc.x = fmaf(s, v.x, acc.x); acc.y = fmaf(s, v.y, acc.y); acc.z = fmaf(s, v.z, acc.z); acc.w = fmaf(s, v.w, acc.w);
}
__device__ __forceinline__ void f4_fma(float4& acc, const float4 a, const float4 v) {
    acc.x = fmaf(a.x, v.x, acc.x); acc.y = fmaf(a.y, v.y, acc.y); acc.z = fmaf(a.z, v.z, acc.z); acc.w = fmaf(a.w, v.w, acc.w);
}
__device__ __forceinline__ float4 f4_mul(const float4 a, const float4 b) {
    return make_float4(a.x * b.x, a.y * b.y, a.z * b.z, a.w * b.w);
}
__device__ __forceinline__ float4 f4_zero() { return make_float4(0.f, 0.f, 0.f, 0.f); }

template <bool IDENT>
__global__ void __launch_bounds__(256, 4)
conv_fwd_kernel(DeviceTables t, Dims dm, int64_t n_nodes, const float* __restrict__ x,
                const float* __restrict__ sh, const float* __restrict__ w,
                const int32_t* __restrict__ senders, const int32_t* __restrict__ rowptr,
                float* __restrict__ out) {
    const int nq4 = dm.nq / 4;
    const int per_node = dm.D * nq4;
    const float4* x4 = reinterpret_cast<const float4*>(x);
    const float4* w4 = reinterpret_cast<const float4*>(w);
    float4* out4 = reinterpret_cast<float4*>(out);
    for (int64_t b = blockIdx.x; b < n_nodes; b += gridDim.x) {
        const int64_t e0 = IDENT ? b : rowptr[b];
        const int64_t e1 = IDENT ? b + 1 : rowptr[b + 1];
        for (int idx = threadIdx.x; idx < per_node; idx += blockDim.x) {
            const int i0 = idx / nq4, q = idx - i0 * nq4;
            const int k = t.i0_path[i0];
            const int r0 = t.i0_start[i0], r1 = t.i0_start[i0 + 1];
            float4 acc = f4_zero();
            int64_t e = e0;
            if (dm.collapsed) {
                // several paths land on this output row: the weight belongs to the record, not to the row
                for (; e < e1; ++e) {
                    const int64_t a = IDENT ? e : (int64_t)senders[e];
                    const float4* xa = x4 + (size_t)a * dm.d * nq4 + q;
                    const float* ye = sh + (size_t)e * dm.dp;
                    const float4* we = w4 + (size_t)e * dm.P * nq4 + q;
                    float4 z = f4_zero();
                    for (int r = r0; r < r1; ++r) {
                        const PackedRecord rc = t.by_i0[r];
                        f4_fma(z, rc.val * ye[rc.b], f4_mul(we[(size_t)rc.c * nq4], xa[(size_t)rc.a * nq4]));
                    }
                    acc.x += z.x; acc.y += z.y; acc.z += z.z; acc.w += z.w;
                }
                out4[((size_t)b * dm.D + i0) * nq4 + q] = acc;
                continue;
            }
            // four edges at a time: their loads are independent and in flight together; the additions stay
            // in edge order
            for (; e + 4 <= e1; e += 4) {
                const float4* xa[4]; const float* ye[4]; float4 we[4], z[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int64_t a = IDENT ? e + u : (int64_t)senders[e + u];
                    xa[u] = x4 + (size_t)a * dm.d * nq4 + q;
                    ye[u] = sh + (size_t)(e + u) * dm.dp;
                    we[u] = w4[((size_t)(e + u) * dm.P + k) * nq4 + q];
                    z[u] = f4_zero();
                }
                for (int r = r0; r < r1; ++r) {
                    const PackedRecord rc = t.by_i0[r];
#pragma unroll
                    for (int u = 0; u < 4; ++u) f4_fma(z[u], rc.val * ye[u][rc.b], xa[u][(size_t)rc.a * nq4]);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) f4_fma(acc, we[u], z[u]);
            }
            for (; e < e1; ++e) {
                const int64_t a = IDENT ? e : (int64_t)senders[e];
                const float4* xa = x4 + (size_t)a * dm.d * nq4 + q;
                const float* ye = sh + (size_t)e * dm.dp;
                float4 z = f4_zero();
                for (int r = r0; r < r1; ++r) {
                    const PackedRecord rc = t.by_i0[r];
                    f4_fma(z, rc.val * ye[rc.b], xa[(size_t)rc.a * nq4]);
                }
                f4_fma(acc, w4[((size_t)e * dm.P + k) * nq4 + q], z);
            }
            out4[((size_t)b * dm.D + i0) * nq4 + q] = acc;
        }
    }
}

// Edge-local cotangents: grad_w[e,k,q] and grad_sh[e,i2]; one block per edge.
template <bool IDENT>
__global__ void __launch_bounds__(256, 4)
conv_bwd_edge_kernel(DeviceTables t, Dims dm, int64_t n_edges, const float* __restrict__ x,
                     const float* __restrict__ sh, const float* __restrict__ w,
                     const int32_t* __restrict__ senders, const int32_t* __restrict__ receivers,
                     const float* __restrict__ g, float* __restrict__ grad_w,
                     float* __restrict__ grad_sh, const int32_t* __restrict__ n_real) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int nq4 = dm.nq / 4;
    // padded call: edges from *n_real on are padding; their gradient rows are zero and nothing of them is read
    const int64_t n_live = n_real ? min((int64_t)*n_real, n_edges) : n_edges;
    for (int64_t e = blockIdx.x; e < n_edges; e += gridDim.x) {
        if (e >= n_live) {
            if (grad_w)
                for (int idx = threadIdx.x; idx < dm.P * dm.nq; idx += blockDim.x)
                    grad_w[(size_t)e * dm.P * dm.nq + idx] = 0.f;
            if (grad_sh && threadIdx.x < dm.dp) grad_sh[(size_t)e * dm.dp + threadIdx.x] = 0.f;
            continue;
        }
        const int64_t a = IDENT ? e : (int64_t)senders[e];
        const int64_t b = IDENT ? e : (int64_t)receivers[e];
        const float4* xa = reinterpret_cast<const float4*>(x) + (size_t)a * dm.d * nq4;
        const float4* gb = reinterpret_cast<const float4*>(g) + (size_t)b * dm.D * nq4;
        const float* ye = sh + (size_t)e * dm.dp;
        const float4* we = reinterpret_cast<const float4*>(w) + (size_t)e * dm.P * nq4;
        if (grad_w) {
            float4* gw4 = reinterpret_cast<float4*>(grad_w) + (size_t)e * dm.P * nq4;
            for (int idx = threadIdx.x; idx < dm.P * nq4; idx += blockDim.x) {
                const int k = idx / nq4, q = idx - k * nq4;
                float4 sum = f4_zero();
                const int row0 = t.path_out_off[k];
                for (int i0 = row0; i0 < row0 + t.path_rows[k]; ++i0) {
                    float4 z = f4_zero();
                    for (int r = t.i0_start[i0]; r < t.i0_start[i0 + 1]; ++r) {
                        const PackedRecord rc = t.by_i0[r];
                        if (rc.c != k) continue;  // (a collapsed plan has other paths' records on this row)
                        f4_fma(z, rc.val * ye[rc.b], xa[(size_t)rc.a * nq4 + q]);
                    }
                    f4_fma(sum, gb[(size_t)i0 * nq4 + q], z);
                }
                gw4[(size_t)k * nq4 + q] = sum;
            }
        }
        if (grad_sh) {
            for (int i2 = warp; i2 < dm.dp; i2 += nwarps) {
                float part = 0.f;
                for (int q = lane; q < nq4; q += 32) {
                    float4 s = f4_zero();
                    for (int r = t.i2_start[i2]; r < t.i2_start[i2 + 1]; ++r) {
                        const PackedRecord rc = t.by_i2[r];  // (i0, i1, path)
                        const float4 wg = f4_mul(we[(size_t)rc.c * nq4 + q], gb[(size_t)rc.a * nq4 + q]);
                        f4_fma(s, f4_mul(make_float4(rc.val, rc.val, rc.val, rc.val), xa[(size_t)rc.b * nq4 + q]), wg);
                    }
                    part += (s.x + s.y) + (s.z + s.w);
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
                if (lane == 0) grad_sh[(size_t)e * dm.dp + i2] = part;
            }
        }
    }
}

// Sender cotangent: grad_x[a,i1,q] gathers over the edges sent by a, in edge order.
template <bool IDENT>
__global__ void __launch_bounds__(256, 4)
conv_bwd_node_kernel(DeviceTables t, Dims dm, int64_t n_nodes, const float* __restrict__ sh,
                     const float* __restrict__ w, const int32_t* __restrict__ receivers,
                     const int32_t* __restrict__ sender_perm, const int32_t* __restrict__ colptr,
                     const float* __restrict__ g, float* __restrict__ grad_x) {
    const int nq4 = dm.nq / 4;
    const int per_node = dm.d * nq4;
    const float4* g4 = reinterpret_cast<const float4*>(g);
    const float4* w4 = reinterpret_cast<const float4*>(w);
    float4* gx4 = reinterpret_cast<float4*>(grad_x);
    for (int64_t a = blockIdx.x; a < n_nodes; a += gridDim.x) {
        const int64_t j0 = IDENT ? a : colptr[a];
        const int64_t j1 = IDENT ? a + 1 : colptr[a + 1];
        for (int idx = threadIdx.x; idx < per_node; idx += blockDim.x) {
            const int i1 = idx / nq4, q = idx - i1 * nq4;
            const int r0 = t.i1_start[i1], r1 = t.i1_start[i1 + 1];
            float4 acc = f4_zero();
            int64_t j = j0;
            // four edges at a time (independent loads in flight together); the additions stay in edge order
            for (; j + 4 <= j1; j += 4) {
                const float4* gb[4]; const float* ye[4]; const float4* we[4]; float4 s4[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int64_t e = IDENT ? j + u : (int64_t)sender_perm[j + u];
                    const int64_t b = IDENT ? e : (int64_t)receivers[e];
                    gb[u] = g4 + (size_t)b * dm.D * nq4 + q;
                    ye[u] = sh + (size_t)e * dm.dp;
                    we[u] = w4 + (size_t)e * dm.P * nq4 + q;
                    s4[u] = f4_zero();
                }
                for (int r = r0; r < r1; ++r) {
                    const PackedRecord rc = t.by_i1[r];  // (i0, i2, path)
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        f4_fma(s4[u], rc.val * ye[u][rc.b],
                               f4_mul(we[u][(size_t)rc.c * nq4], gb[u][(size_t)rc.a * nq4]));
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) { acc.x += s4[u].x; acc.y += s4[u].y; acc.z += s4[u].z; acc.w += s4[u].w; }
            }
            for (; j < j1; ++j) {
                const int64_t e = IDENT ? j : (int64_t)sender_perm[j];
                const int64_t b = IDENT ? e : (int64_t)receivers[e];
                const float4* gb = g4 + (size_t)b * dm.D * nq4 + q;
                const float* ye = sh + (size_t)e * dm.dp;
                const float4* we = w4 + (size_t)e * dm.P * nq4 + q;
                float4 s = f4_zero();
                for (int r = r0; r < r1; ++r) {
                    const PackedRecord rc = t.by_i1[r];  // (i0, i2, path)
                    f4_fma(s, rc.val * ye[rc.b], f4_mul(we[(size_t)rc.c * nq4], gb[(size_t)rc.a * nq4]));
                }
                acc.x += s.x; acc.y += s.y; acc.z += s.z; acc.w += s.w;
            }
            gx4[((size_t)a * dm.d + i1) * nq4 + q] = acc;
        }
    }
}

}  // namespace generic
}  // namespace e3j
