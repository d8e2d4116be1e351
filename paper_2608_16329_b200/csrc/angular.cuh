// Angular bases beyond the default closed forms (fp64 path): the canonical basis of all Cartesian monomials up to
// l_max (Section 3.3, Eq. 11: d = 1, 4, 10, 20, ...) with the metric C_l = multinomial multiplicities of Eq. 5, and
// the irreducible basis for l_max = 4, 5 (d = 25, 36) through projection matrices Q_l (Section 3.3.1) that the host
// constructs once and places in constant memory.  Monomials of a degree are ordered by descending power of x, then of y
// (x^2, xy, xz, y^2, yz, z^2), as in the text below Eq. 11.
#pragma once
#include "common.cuh"

namespace mlip {

constexpr int ANG_LMAX = 5;
__host__ __device__ constexpr int n_mono(int l) { return (l + 1) * (l + 2) / 2; }
__host__ __device__ constexpr int q_offset(int l) {   // start of Q_l in the concatenation Q_0, Q_1, ...
    int o = 0;
    for (int m = 0; m < l; ++m) o += (2 * m + 1) * n_mono(m);
    return o;
}
constexpr int Q_TOTAL = q_offset(ANG_LMAX + 1);   // 476 entries for l <= 5
__host__ __device__ constexpr int factorial_i(int n) { int f = 1; for (int q = 2; q <= n; ++q) f *= q; return f; }

template <int LMAX, int BASIS>
struct AngShape {
    static_assert(LMAX >= 0 && LMAX <= ANG_LMAX && (BASIS == 0 || BASIS == 1), "angular shape not compiled in");
    __host__ __device__ static constexpr int rows(int l) { return BASIS ? n_mono(l) : 2 * l + 1; }
    __host__ __device__ static constexpr int begin(int l) { int o = 0; for (int m = 0; m < l; ++m) o += rows(m); return o; }
    static constexpr int D = begin(LMAX + 1);
    __host__ __device__ static constexpr int l_of(int a) { int l = 0; while (begin(l + 1) <= a) ++l; return l; }
    // diagonal entry of C_l for row a: 1 for the orthonormal irreducible rows, l! / (ax! ay! az!) for monomial rows
    __host__ __device__ static constexpr double metric(int a) {
        if (!BASIS) return 1.0;
        const int l = l_of(a);
        int c = a - begin(l), idx = 0;
        for (int ax = l; ax >= 0; --ax)
            for (int ay = l - ax; ay >= 0; --ay) {
                if (idx == c) return (double)factorial_i(l) / (double)(factorial_i(ax) * factorial_i(ay) * factorial_i(l - ax - ay));
                ++idx;
            }
        return 1.0;
    }
};

// Q_0 .. Q_5 (irreducible projections) in constant memory; every access in the kernels is warp-uniform.  The array is
// private to the translation unit that includes this header for device code (the fp64 kernel), which also fills it.
static __constant__ double c_ang_q[Q_TOTAL];

// Host (angular.cu): Q_0 .. Q_5 concatenated row-major, Q_TOTAL doubles.
void build_q_tables(double *out);

// h = angular feature vector of the unit vector (x, y, z).
template <int LMAX, int BASIS>
__device__ __forceinline__ void angular_values(double x, double y, double z, double *h) {
    using S = AngShape<LMAX, BASIS>;
    double px[LMAX + 1], py[LMAX + 1], pz[LMAX + 1];
    px[0] = py[0] = pz[0] = 1.0;
#pragma unroll
    for (int q = 1; q <= LMAX; ++q) { px[q] = px[q - 1] * x; py[q] = py[q - 1] * y; pz[q] = pz[q - 1] * z; }
#pragma unroll
    for (int l = 0; l <= LMAX; ++l) {
        if (!BASIS) {
#pragma unroll
            for (int r = 0; r < 2 * l + 1; ++r) h[S::begin(l) + r] = 0.0;
        }
        int c = 0;
#pragma unroll
        for (int ax = l; ax >= 0; --ax)
#pragma unroll
            for (int ay = l - ax; ay >= 0; --ay) {
                const double m = px[ax] * py[ay] * pz[l - ax - ay];
                if (BASIS) h[S::begin(l) + c] = m;
                else {
#pragma unroll
                    for (int r = 0; r < 2 * l + 1; ++r) h[S::begin(l) + r] = fma(c_ang_q[q_offset(l) + r * n_mono(l) + c], m, h[S::begin(l) + r]);
                }
                ++c;
            }
    }
}

// s = sum_a h_a t_a,  (tx, ty, tz) = sum_a v_a grad h_a,  tu = u . (tx, ty, tz)  (= sum_a l_a v_a h_a by Euler's theorem).
// v and t are first brought to monomial coefficients (Q_l^T v, Q_l^T t; the identity for the canonical basis).
// Only the degrees L0 .. L1 are taken, with v and t holding the rows of those degrees (v[0] = first row of degree L0):
// the sums are linear in v and t, so a caller short of registers adds the results of several degree ranges.
template <int LMAX, int BASIS, int L0 = 0, int L1 = LMAX>
__device__ __forceinline__ void angular_project(double x, double y, double z, const double *v, const double *t, double &s, double &tx,
                                                double &ty, double &tz, double &tu) {
    using S = AngShape<LMAX, BASIS>;
    double px[LMAX + 1], py[LMAX + 1], pz[LMAX + 1];
    px[0] = py[0] = pz[0] = 1.0;
#pragma unroll
    for (int q = 1; q <= LMAX; ++q) { px[q] = px[q - 1] * x; py[q] = py[q - 1] * y; pz[q] = pz[q - 1] * z; }
    double acc = 0.0, gx = 0.0, gy = 0.0, gz = 0.0;
    constexpr int row0 = S::begin(L0);
#pragma unroll
    for (int l = L0; l <= L1; ++l) {
        int c = 0;
#pragma unroll
        for (int ax = l; ax >= 0; --ax)
#pragma unroll
            for (int ay = l - ax; ay >= 0; --ay) {
                const int az = l - ax - ay;
                double vc, tc;
                if (BASIS) { vc = v[S::begin(l) - row0 + c]; tc = t[S::begin(l) - row0 + c]; }
                else {
                    vc = 0.0; tc = 0.0;
#pragma unroll
                    for (int r = 0; r < 2 * l + 1; ++r) {
                        const double q = c_ang_q[q_offset(l) + r * n_mono(l) + c];
                        vc = fma(q, v[S::begin(l) - row0 + r], vc);
                        tc = fma(q, t[S::begin(l) - row0 + r], tc);
                    }
                }
                acc = fma(tc, px[ax] * py[ay] * pz[az], acc);
                if (ax > 0) gx = fma(vc * (double)ax, px[ax - 1] * py[ay] * pz[az], gx);
                if (ay > 0) gy = fma(vc * (double)ay, px[ax] * py[ay - 1] * pz[az], gy);
                if (az > 0) gz = fma(vc * (double)az, px[ax] * py[ay] * pz[az - 1], gz);
                ++c;
            }
    }
    s = acc; tx = gx; ty = gy; tz = gz;
    tu = x * gx + y * gy + z * gz;
}


}  // namespace mlip
