// Real spherical harmonics of an edge direction, l <= 3 (paper, "Key Operations in Scope": the harmonic embedding
// Y(r_ab / |r_ab|) that the convolution takes as y).  Component normalisation (sum over m of Y_lm^2 = 2l+1 on the
// unit sphere, Y_0 = 1), degrees stacked l = 0..lmax with m = -l..l inside a degree: l = 1 is sqrt(3) (y, z, x).
// Cartesian closed forms of the unit vector; the gradient is that of the polynomials as written, which the
// caller projects onto the tangent plane (Y depends on the direction only).
#pragma once

namespace e3j {
namespace fast {

// unit vector of v; a zero vector has no direction: it maps to (0, 0, 0) and inv_r = 0
__device__ __forceinline__ void unit_vector(float vx, float vy, float vz, float& x, float& y, float& z, float& inv_r) {
    const float r2 = fmaf(vx, vx, fmaf(vy, vy, vz * vz));
    inv_r = r2 > 0.f ? rsqrtf(r2) : 0.f;
    // one Newton step: rsqrtf alone is 2 ulp, the harmonics should be as good as float32 inputs allow
    inv_r = inv_r * fmaf(-0.5f * r2 * inv_r, inv_r, 1.5f);
    x = vx * inv_r; y = vy * inv_r; z = vz * inv_r;
}

// Y[0 .. DSH) for DSH = (lmax + 1)^2 in {1, 4, 9, 16}
template <int DSH>
__device__ __forceinline__ void harmonics(const float x, const float y, const float z, float (&Y)[DSH]) {
    static_assert(DSH == 1 || DSH == 4 || DSH == 9 || DSH == 16, "closed forms are written out for l <= 3");
    Y[0] = 1.f;
    if constexpr (DSH >= 4) {
        constexpr float r3 = 1.7320508075688772f;
        Y[1] = r3 * y; Y[2] = r3 * z; Y[3] = r3 * x;
    }
    if constexpr (DSH >= 9) {
        constexpr float r15 = 3.872983346207417f, r5h = 1.118033988749895f;   // sqrt(15), sqrt(5) / 2
        Y[4] = r15 * x * y;
        Y[5] = r15 * y * z;
        Y[6] = r5h * fmaf(3.f * z, z, -1.f);
        Y[7] = r15 * x * z;
        Y[8] = 0.5f * r15 * (x * x - y * y);
    }
    if constexpr (DSH >= 16) {
        constexpr float a = 2.091650066335189f;    // sqrt(35 / 8)
        constexpr float b = 10.246950765959598f;   // sqrt(105)
        constexpr float c = 1.620185174601965f;    // sqrt(21 / 8)
        constexpr float r7h = 1.3228756555322954f; // sqrt(7) / 2
        const float x2 = x * x, y2 = y * y, z2 = z * z;
        Y[9] = a * y * (3.f * x2 - y2);
        Y[10] = b * x * y * z;
        Y[11] = c * y * fmaf(5.f, z2, -1.f);
        Y[12] = r7h * z * fmaf(5.f, z2, -3.f);
        Y[13] = c * x * fmaf(5.f, z2, -1.f);
        Y[14] = 0.5f * b * (x2 - y2) * z;
        Y[15] = a * x * (x2 - 3.f * y2);
    }
}

// (gx, gy, gz) = sum_i g[i] * grad Y_i at the unit vector (x, y, z): gradient of the polynomials above
template <int DSH>
__device__ __forceinline__ void harmonics_vjp(const float x, const float y, const float z, const float (&g)[DSH],
                                              float& gx, float& gy, float& gz) {
    gx = gy = gz = 0.f;
    if constexpr (DSH >= 4) {
        constexpr float r3 = 1.7320508075688772f;
        gy = r3 * g[1]; gz = r3 * g[2]; gx = r3 * g[3];
    }
    if constexpr (DSH >= 9) {
        constexpr float r15 = 3.872983346207417f, r5h = 1.118033988749895f;
        gx += r15 * (g[4] * y + g[7] * z + g[8] * x);
        gy += r15 * (g[4] * x + g[5] * z - g[8] * y);
        gz += r15 * (g[5] * y + g[7] * x) + 6.f * r5h * g[6] * z;
    }
    if constexpr (DSH >= 16) {
        constexpr float a = 2.091650066335189f, b = 10.246950765959598f, c = 1.620185174601965f;
        constexpr float r7h = 1.3228756555322954f;
        const float x2 = x * x, y2 = y * y, z2 = z * z;
        const float q = fmaf(5.f, z2, -1.f);
        gx += a * (g[9] * 6.f * x * y + g[15] * 3.f * (x2 - y2)) + b * (g[10] * y * z + g[14] * x * z) + c * g[13] * q;
        gy += a * (g[9] * 3.f * (x2 - y2) - g[15] * 6.f * x * y) + b * (g[10] * x * z - g[14] * y * z) + c * g[11] * q;
        gz += b * (g[10] * x * y + 0.5f * g[14] * (x2 - y2)) + 10.f * c * z * (g[11] * y + g[13] * x)
              + r7h * g[12] * fmaf(15.f, z2, -3.f);
    }
}

}  // namespace fast
}  // namespace e3j
