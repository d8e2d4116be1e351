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

// s = sum_a h_a t_a,  (tx,ty,tz) = sum_a v_a grad h_a,  tu = sum_a l_a v_a h_a  (Euler: grad h_a . u = l_a h_a).
template <typename T>
__device__ __forceinline__ void harmonics_project(T x, T y, T z, const T *v, const T *t, T &s, T &tx, T &ty, T &tz, T &tu) {
    const T s2 = T(1.4142135623730951), is2 = T(0.7071067811865476), is6 = T(0.4082482904638631);
    const T s6 = T(2.449489742783178), s15 = T(1.224744871391589), is10 = T(0.31622776601683794);
    T xx = x * x, yy = y * y, zz = z * z, h;
    s = t[0]; tx = ty = tz = T(0); tu = T(0);
    s += x * t[1] + y * t[2] + z * t[3];
    tx += v[1]; ty += v[2]; tz += v[3];
    tu += x * v[1] + y * v[2] + z * v[3];
    T u2 = T(0);
    h = s2 * x * y; s += h * t[4]; u2 += h * v[4]; tx += s2 * y * v[4]; ty += s2 * x * v[4];
    h = s2 * x * z; s += h * t[5]; u2 += h * v[5]; tx += s2 * z * v[5]; tz += s2 * x * v[5];
    h = s2 * y * z; s += h * t[6]; u2 += h * v[6]; ty += s2 * z * v[6]; tz += s2 * y * v[6];
    h = is2 * (xx - yy); s += h * t[7]; u2 += h * v[7]; tx += s2 * x * v[7]; ty -= s2 * y * v[7];
    h = is6 * (T(2) * zz - xx - yy); s += h * t[8]; u2 += h * v[8];
    tx -= T(2) * is6 * x * v[8]; ty -= T(2) * is6 * y * v[8]; tz += T(4) * is6 * z * v[8];
    T u3 = T(0);
    h = s6 * x * y * z; s += h * t[9]; u3 += h * v[9];
    tx += s6 * y * z * v[9]; ty += s6 * x * z * v[9]; tz += s6 * x * y * v[9];
    h = s15 * z * (xx - yy); s += h * t[10]; u3 += h * v[10];
    tx += T(2) * s15 * x * z * v[10]; ty -= T(2) * s15 * y * z * v[10]; tz += s15 * (xx - yy) * v[10];
    h = s15 * x * (yy - zz); s += h * t[11]; u3 += h * v[11];
    tx += s15 * (yy - zz) * v[11]; ty += T(2) * s15 * x * y * v[11]; tz -= T(2) * s15 * x * z * v[11];
    h = s15 * y * (zz - xx); s += h * t[12]; u3 += h * v[12];
    tx -= T(2) * s15 * x * y * v[12]; ty += s15 * (zz - xx) * v[12]; tz += T(2) * s15 * y * z * v[12];
    h = is10 * x * (T(2) * xx - T(3) * yy - T(3) * zz); s += h * t[13]; u3 += h * v[13];
    tx += is10 * (T(6) * xx - T(3) * yy - T(3) * zz) * v[13]; ty -= T(6) * is10 * x * y * v[13]; tz -= T(6) * is10 * x * z * v[13];
    h = is10 * y * (T(2) * yy - T(3) * xx - T(3) * zz); s += h * t[14]; u3 += h * v[14];
    tx -= T(6) * is10 * x * y * v[14]; ty += is10 * (T(6) * yy - T(3) * xx - T(3) * zz) * v[14]; tz -= T(6) * is10 * y * z * v[14];
    h = is10 * z * (T(2) * zz - T(3) * xx - T(3) * yy); s += h * t[15]; u3 += h * v[15];
    tx -= T(6) * is10 * x * z * v[15]; ty -= T(6) * is10 * y * z * v[15]; tz += is10 * (T(6) * zz - T(3) * xx - T(3) * yy) * v[15];
    tu += T(2) * u2 + T(3) * u3;
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
