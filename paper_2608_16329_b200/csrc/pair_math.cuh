// Per-pair math shared by the fp32/tensor-pipe kernel and the fp64 kernel: irreducible harmonics
// (Eq. 3), their projection onto the pair vector (Eq. 10), the cubic B-spline basis of the radial
// tables (Eq. 2) and SiLU.  Templated on the scalar type.
#pragma once
#include "common.cuh"

namespace mlip {

// Irreducible harmonic polynomials up to l = 3 of a unit vector (one valid solution of the
// projection constraints of Section 3.3.1: harmonic, orthonormal under the multinomial metric).
template <typename T>
__device__ __forceinline__ void harmonics(T x, T y, T z, T *h) {
    const T s2 = T(1.4142135623730951), is2 = T(0.7071067811865476), is6 = T(0.4082482904638631);
    const T s6 = T(2.449489742783178), s15 = T(1.224744871391589), is10 = T(0.31622776601683794);
    T xx = x * x, yy = y * y, zz = z * z;
    h[0] = T(1);
    h[1] = x; h[2] = y; h[3] = z;
    h[4] = s2 * x * y; h[5] = s2 * x * z; h[6] = s2 * y * z;
    h[7] = is2 * (xx - yy);
    h[8] = is6 * (T(2) * zz - xx - yy);
    h[9] = s6 * x * y * z;
    h[10] = s15 * z * (xx - yy);
    h[11] = s15 * x * (yy - zz);
    h[12] = s15 * y * (zz - xx);
    h[13] = is10 * x * (T(2) * xx - T(3) * yy - T(3) * zz);
    h[14] = is10 * y * (T(2) * yy - T(3) * xx - T(3) * zz);
    h[15] = is10 * z * (T(2) * zz - T(3) * xx - T(3) * yy);
}

// s = sum_a h_a t_a,  (tx,ty,tz) = sum_a v_a grad h_a,  tu = sum_a l_a v_a h_a.
// The gradient is taken of the polynomial Phi(u) = sum_a v_a h_a(u): its quadratic and cubic parts are written out in
// monomial coefficients (a fixed linear map of v), which costs fewer operations than seven separate gradients, and
// tu = u . grad Phi by Euler's theorem for homogeneous polynomials (grad h_a . u = l_a h_a).  (x, y, z) is a unit vector;
// the values h_a in s use x^2 + y^2 + z^2 = 1 where that shortens them.
template <typename T>
__device__ __forceinline__ void harmonics_project(T x, T y, T z, const T *v, const T *t, T &s, T &tx, T &ty, T &tz, T &tu) {
    const T s2 = T(1.4142135623730951), is2 = T(0.7071067811865476), is6 = T(0.4082482904638631);
    const T s6 = T(2.449489742783178), s15 = T(1.224744871391589), is10 = T(0.31622776601683794);
    const T xx = x * x, yy = y * y, zz = z * z, xy = x * y, xz = x * z, yz = y * z;
    // ---- s: the harmonics' values against t
    const T dxy = xx - yy, dyz = yy - zz, dzx = zz - xx;
    T acc = t[0] + x * t[1] + y * t[2] + z * t[3];
    acc += s2 * (xy * t[4] + xz * t[5] + yz * t[6]) + is2 * (dxy * t[7]) + is6 * ((T(3) * zz - T(1)) * t[8]);
    acc += s6 * (xy * (z * t[9])) + s15 * (z * dxy * t[10] + x * dyz * t[11] + y * dzx * t[12]);
    acc += is10 * (x * (T(5) * xx - T(3)) * t[13] + y * (T(5) * yy - T(3)) * t[14] + z * (T(5) * zz - T(3)) * t[15]);
    s = acc;
    // ---- quadratic part: Phi_2 = (Bxx x^2 + Byy y^2 + Bzz z^2) / 2 + Axy xy + Axz xz + Ayz yz
    const T axy = s2 * v[4], axz = s2 * v[5], ayz = s2 * v[6], w7 = s2 * v[7], w8 = (T(2) * is6) * v[8];
    const T bxx = w7 - w8, byy = -w7 - w8, bzz = T(2) * w8;
    T gx = v[1] + bxx * x + axy * y + axz * z;
    T gy = v[2] + axy * x + byy * y + ayz * z;
    T gz = v[3] + axz * x + ayz * y + bzz * z;
    // ---- cubic part: Phi_3 = (2/3)(p13 x^3 + p14 y^3 + p15 z^3) + x (cxyy y^2 + cxzz z^2) + y (cyxx x^2 + cyzz z^2)
    //                          + z (czxx x^2 + czyy y^2) + cxyz xyz,   p = 3 v / sqrt(10), q = sqrt(3/2) v
    const T p13 = (T(3) * is10) * v[13], p14 = (T(3) * is10) * v[14], p15 = (T(3) * is10) * v[15];
    const T q10 = s15 * v[10], q11 = s15 * v[11], q12 = s15 * v[12], cxyz = s6 * v[9];
    const T cxyy = q11 - p13, cxzz = -q11 - p13, cyxx = -q12 - p14, cyzz = q12 - p14, czxx = q10 - p15, czyy = -q10 - p15;
    const T x2 = x + x, y2 = y + y, z2 = z + z;
    gx += p13 * (xx + xx) + cxyy * yy + cxzz * zz + x2 * (cyxx * y + czxx * z) + cxyz * yz;
    gy += p14 * (yy + yy) + cyxx * xx + cyzz * zz + y2 * (cxyy * x + czyy * z) + cxyz * xz;
    gz += p15 * (zz + zz) + czxx * xx + czyy * yy + z2 * (cxzz * x + cyzz * y) + cxyz * xy;
    tx = gx; ty = gy; tz = gz;
    tu = x * gx + y * gy + z * gz;
}

// Spline interval and cubic B-spline basis (and its r-derivative) at distance r for a table of
// `knots` intervals of width 1 / inv_h starting at r_min.
template <bool DERIV, typename T>
__device__ __forceinline__ int spline_basis(T r, T r_min, T inv_h, int knots, T *b, T *db, int *status) {
    T xk = (r - r_min) * inv_h;
    if (xk < T(0)) { atomicOr(status, FLAG_TABLE_RANGE); xk = T(0); }
    int i = (int)xk;
    i = i > knots - 1 ? knots - 1 : i;
    T u = xk - (T)i, u2 = u * u, u3 = u2 * u, w = T(1) - u;
    const T sixth = T(1) / T(6);
    b[0] = w * w * w * sixth;
    b[1] = (T(3) * u3 - T(6) * u2 + T(4)) * sixth;
    b[2] = (T(-3) * u3 + T(3) * u2 + T(3) * u + T(1)) * sixth;
    b[3] = u3 * sixth;
    if (DERIV) {
        db[0] = T(-0.5) * w * w * inv_h;
        db[1] = (T(1.5) * u2 - T(2) * u) * inv_h;
        db[2] = (T(-1.5) * u2 + u + T(0.5)) * inv_h;
        db[3] = T(0.5) * u2 * inv_h;
    }
    return i;
}

}  // namespace mlip
