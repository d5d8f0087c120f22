// Test infrastructure: lets the generated per-edge bodies of the specialised kernels (the `struct Sig_<name>` part
// of csrc/fast/sig_<name>.cu) be compiled for the host, one lane at a time, so that the generator's output can be
// checked against the oracle without a GPU.  Nothing of the product includes this file.
//
// Part 1 (before the generated text): the handful of vector types and helpers the bodies use.
// Part 2 (after it, E3J_HOST_RUNNERS defined): runners that do for one edge what the kernels' warps do around the
// bodies: contract the A entries from the harmonics with the slot tables, call the body for every lane, and put
// the lanes' results together.
#ifndef E3J_HOST_RUNNERS
#include <cmath>
#include <cstdint>
#include <cstring>

#define __device__
#define __forceinline__ inline
#define __restrict__

struct float2 { float x, y; };
struct float4 { float x, y, z, w; };
inline float2 make_float2(float x, float y) { return float2{x, y}; }
inline float4 make_float4(float x, float y, float z, float w) { return float4{x, y, z, w}; }

namespace e3j {
namespace fast {
struct PairRec { int16_t start, count; };

inline float4 vmul(const float4 a, const float4 b) { return make_float4(a.x * b.x, a.y * b.y, a.z * b.z, a.w * b.w); }
inline float2 vmul(const float2 a, const float2 b) { return make_float2(a.x * b.x, a.y * b.y); }
inline float vmul(const float a, const float b) { return a * b; }
inline void vfma(float4& acc, const float a, const float4 b) {
    acc.x = fmaf(a, b.x, acc.x); acc.y = fmaf(a, b.y, acc.y); acc.z = fmaf(a, b.z, acc.z); acc.w = fmaf(a, b.w, acc.w);
}
inline void vfma(float2& acc, const float a, const float2 b) { acc.x = fmaf(a, b.x, acc.x); acc.y = fmaf(a, b.y, acc.y); }
inline void vfma(float4& acc, const float4 a, const float4 b) {
    acc.x = fmaf(a.x, b.x, acc.x); acc.y = fmaf(a.y, b.y, acc.y); acc.z = fmaf(a.z, b.z, acc.z); acc.w = fmaf(a.w, b.w, acc.w);
}
inline void vfma(float2& acc, const float2 a, const float2 b) { acc.x = fmaf(a.x, b.x, acc.x); acc.y = fmaf(a.y, b.y, acc.y); }
inline void vfma(float& acc, const float a, const float b) { acc = fmaf(a, b, acc); }
// the packed forms of the device code compute the same IEEE operations
template <class A, class B> inline auto pmul(const A a, const B b) { return vmul(a, b); }
template <class V, class A, class B> inline void pfma(V& acc, const A a, const B b) { vfma(acc, a, b); }
inline float vdot(const float4 a, const float4 b) { return fmaf(a.w, b.w, fmaf(a.z, b.z, fmaf(a.y, b.y, a.x * b.x))); }
inline float vdot(const float2 a, const float2 b) { return fmaf(a.y, b.y, a.x * b.x); }
inline float vdot(const float a, const float b) { return a * b; }
inline void vzero(float4& v) { v = make_float4(0.f, 0.f, 0.f, 0.f); }
inline void vzero(float2& v) { v = make_float2(0.f, 0.f); }
inline void vzero(float& v) { v = 0.f; }
}  // namespace fast
}  // namespace e3j

#else  // ------------------------------------------------------------------ part 2: runners
namespace host_run {

template <class VecT> constexpr int width() { return (int)(sizeof(VecT) / sizeof(float)); }

// A[slot] = sum over the slot's records of c * y[i2] (what the producer warps compute per edge)
template <class PairFn, class ValFn, class I2Fn>
inline void contract_A(int n_slots, PairFn pair, ValFn val, I2Fn i2, const float* y, float* A) {
    for (int s = 0; s < n_slots; ++s) {
        const auto pr = pair(s);
        float a = 0.f;
        for (int j = 0; j < pr.count; ++j) a += val(pr.start + j) * y[i2(pr.start + j)];
        A[s] = a;
    }
}

template <class S, int G>
struct FwdGroups {
    static void run(const float* x, const float* s, const float* A, float* out, int lane) {
        using Vec = typename S::Vec;
        constexpr int V = S::V, NQV = S::NQ / V;
        Vec acc[S::F_RMAX];
        std::memset(acc, 0, sizeof(acc));
        S::template fwd_edge<G>(acc, reinterpret_cast<const Vec*>(x) + lane, reinterpret_cast<const Vec*>(s) + lane, A);
        for (int row = S::f_row0(G); row < S::f_row0(G + 1); ++row)
            std::memcpy(out + (size_t)row * S::NQ + lane * V, &acc[row - S::f_row0(G)], sizeof(Vec));
        (void)NQV;
        FwdGroups<S, G + 1>::run(x, s, A, out, lane);
    }
};
template <class S>
struct FwdGroups<S, S::FW> {
    static void run(const float*, const float*, const float*, float*, int) {}
};

// out[D][NQ] of one edge (the forward's per-receiver sum has a single term)
template <class S>
void fwd(const float* x, const float* y, const float* s, float* out) {
    alignas(16) float A[S::F_APAD + 4];
    contract_A(S::F_APAD, [](int i) { return S::pair_rec(i); }, [](int i) { return S::rec_val(i); },
               [](int i) { return S::rec_i2(i); }, y, A);
    for (int lane = 0; lane < S::NQ / S::V; ++lane) FwdGroups<S, 0>::run(x, s, A, out, lane);
}

template <class S>
void bwd_tables(const float* y, float* A) {
    contract_A(S::B_APAD, [](int i) { return S::b_pair_rec(i); }, [](int i) { return S::b_rec_val(i); },
               [](int i) { return S::b_rec_i2(i); }, y, A);
}

// path-group backward: every group's partial sums added in group order, as the kernel's exchange does
template <class S>
void bwd_groups(const float* x, const float* y, const float* s, const float* g, float* dx, float* dy, float* ds) {
    using Vec = typename S::BVec;
    constexpr int V = S::BV, NQV = S::NQ / V;
    alignas(16) float A[S::B_APAD + 4];
    bwd_tables<S>(y, A);
    for (int i = 0; i < S::DSH; ++i) dy[i] = 0.f;
    for (int i = 0; i < S::DIN * S::NQ; ++i) dx[i] = 0.f;
    for (int lane = 0; lane < NQV; ++lane) {
        for (int G = 0; G < S::BW; ++G) {
            Vec dm[S::B_RMAX];
            std::memset(dm, 0, sizeof(dm));
            for (int r = 0; r < S::b_nrow(G); ++r)
                std::memcpy(&dm[r], g + (size_t)S::b_row(G, r) * S::NQ + lane * V, sizeof(Vec));
            Vec dxp[S::DIN];
            float dyl[16];
            S::bwd_edge(G, dm, reinterpret_cast<const Vec*>(x) + lane, reinterpret_cast<const Vec*>(s) + lane, A, dxp,
                        dyl, reinterpret_cast<Vec*>(ds) + lane);
            for (int i = 0; i < S::DIN; ++i)
                for (int c = 0; c < V; ++c) dx[(size_t)i * S::NQ + lane * V + c] += reinterpret_cast<const float*>(&dxp[i])[c];
            for (int i = 0; i < S::DSH; ++i) dy[i] += dyl[i];
        }
    }
}

// edge-wise backward: one call per lane yields everything
template <class S>
void bwd_all(const float* x, const float* y, const float* s, const float* g, float* dx, float* dy, float* ds) {
    if constexpr (S::ET > 0 || S::ETR > 0) {
        using Vec = typename S::EVec;
        constexpr int V = S::EV, NQV = S::NQ / V;
        alignas(16) float A[S::B_APAD + 4];
        bwd_tables<S>(y, A);
        for (int i = 0; i < S::DSH; ++i) dy[i] = 0.f;
        for (int lane = 0; lane < NQV; ++lane) {
            Vec dxp[S::DIN];
            float dyl[16];
            S::bwd_edge_all(reinterpret_cast<const Vec*>(g) + lane, reinterpret_cast<const Vec*>(x) + lane,
                            reinterpret_cast<const Vec*>(s) + lane, A, dxp, dyl, reinterpret_cast<Vec*>(ds) + lane);
            for (int i = 0; i < S::DIN; ++i) std::memcpy(dx + (size_t)i * S::NQ + lane * V, &dxp[i], sizeof(Vec));
            for (int i = 0; i < S::DSH; ++i) dy[i] += dyl[i];
        }
    }
}

template <class S, int G>
struct Fwd2Groups {
    static void run(const float* x, const float* ux, const float* s, const float* us, const float* A, const float* B,
                    float* out, int lane) {
        using Vec = typename S::DFVec;
        constexpr int V = S::DFV;
        Vec acc[S::F_RMAX];
        std::memset(acc, 0, sizeof(acc));
        S::template fwd2_edge<G>(acc, reinterpret_cast<const Vec*>(x) + lane, reinterpret_cast<const Vec*>(ux) + lane,
                                 reinterpret_cast<const Vec*>(s) + lane, reinterpret_cast<const Vec*>(us) + lane, A, B);
        for (int row = S::f_row0(G); row < S::f_row0(G + 1); ++row)
            std::memcpy(out + (size_t)row * S::NQ + lane * V, &acc[row - S::f_row0(G)], sizeof(Vec));
        Fwd2Groups<S, G + 1>::run(x, ux, s, us, A, B, out, lane);
    }
};
template <class S>
struct Fwd2Groups<S, S::FW> {
    static void run(const float*, const float*, const float*, const float*, const float*, const float*, float*, int) {}
};

// double backward of one edge: cotangent of grad_out (forward-shaped) and cotangents of x, sh, w (edge sweep)
template <class S>
void dbl(const float* x, const float* y, const float* s, const float* g, const float* ux, const float* uy,
         const float* us, float* gg, float* dx, float* dy, float* ds) {
    if constexpr (S::DFT > 0) {
        alignas(16) float A[S::F_APAD + 4], B[S::F_APAD + 4];
        contract_A(S::F_APAD, [](int i) { return S::pair_rec(i); }, [](int i) { return S::rec_val(i); },
                   [](int i) { return S::rec_i2(i); }, y, A);
        contract_A(S::F_APAD, [](int i) { return S::pair_rec(i); }, [](int i) { return S::rec_val(i); },
                   [](int i) { return S::rec_i2(i); }, uy, B);
        for (int lane = 0; lane < S::NQ / S::DFV; ++lane) Fwd2Groups<S, 0>::run(x, ux, s, us, A, B, gg, lane);
    }
    if constexpr (S::DT > 0) {
        using Vec = typename S::DVec;
        constexpr int V = S::DV, NQV = S::NQ / V;
        alignas(16) float A[S::B_APAD + 4], B[S::B_APAD + 4];
        bwd_tables<S>(y, A);
        bwd_tables<S>(uy, B);
        for (int i = 0; i < S::DSH; ++i) dy[i] = 0.f;
        for (int lane = 0; lane < NQV; ++lane) {
            Vec dxp[S::DIN];
            float dyl[16];
            S::bwd2_edge_all(reinterpret_cast<const Vec*>(g) + lane, reinterpret_cast<const Vec*>(x) + lane,
                             reinterpret_cast<const Vec*>(ux) + lane, reinterpret_cast<const Vec*>(s) + lane,
                             reinterpret_cast<const Vec*>(us) + lane, A, B, dxp, dyl, reinterpret_cast<Vec*>(ds) + lane);
            for (int i = 0; i < S::DIN; ++i) std::memcpy(dx + (size_t)i * S::NQ + lane * V, &dxp[i], sizeof(Vec));
            for (int i = 0; i < S::DSH; ++i) dy[i] += dyl[i];
        }
    }
}

}  // namespace host_run
#endif
