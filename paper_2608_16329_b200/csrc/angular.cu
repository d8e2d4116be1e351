// Host-side construction of the irreducible projection matrices Q_l (Section 3.3.1) for l <= 5.
// Q_l has 2l + 1 rows over the C(l+2, 2) monomials of degree l and satisfies the two constraints of the paper:
//   L_l Q_l^T = 0            every row is a harmonic polynomial (L_l = the Laplacian on degree-l coefficients)
//   Q_l D_l^{-1} Q_l^T = I   rows orthonormal under the metric 1 / D_l, D_l = l! / (ax! ay! az!)
// Construction: a basis of the null space of L_l by elimination, then Gram-Schmidt under that metric.  Q_l is fixed only
// up to an orthogonal mixing of its rows; the invariants of Eq. 5 do not depend on the choice.
#include <math.h>
#include <vector>

#include "angular.cuh"

namespace mlip {

namespace {

struct Exps { int ax, ay, az; };

std::vector<Exps> monomials(int l) {
    std::vector<Exps> e;
    for (int ax = l; ax >= 0; --ax)
        for (int ay = l - ax; ay >= 0; --ay) e.push_back({ax, ay, l - ax - ay});
    return e;
}

int find(const std::vector<Exps> &e, int ax, int ay, int az) {
    for (size_t q = 0; q < e.size(); ++q)
        if (e[q].ax == ax && e[q].ay == ay && e[q].az == az) return (int)q;
    return -1;
}

// rows of the null space of the Laplacian on degree-l coefficient vectors
std::vector<std::vector<double>> harmonic_basis(int l) {
    const std::vector<Exps> src = monomials(l);
    const int n = (int)src.size();
    std::vector<std::vector<double>> basis;
    if (l < 2) {
        for (int q = 0; q < n; ++q) { std::vector<double> v(n, 0.0); v[q] = 1.0; basis.push_back(v); }
        return basis;
    }
    const std::vector<Exps> dst = monomials(l - 2);
    const int m = (int)dst.size();
    std::vector<std::vector<double>> L(m, std::vector<double>(n, 0.0));
    for (int col = 0; col < n; ++col) {
        const Exps &e = src[col];
        if (e.ax >= 2) L[find(dst, e.ax - 2, e.ay, e.az)][col] += e.ax * (e.ax - 1);
        if (e.ay >= 2) L[find(dst, e.ax, e.ay - 2, e.az)][col] += e.ay * (e.ay - 1);
        if (e.az >= 2) L[find(dst, e.ax, e.ay, e.az - 2)][col] += e.az * (e.az - 1);
    }
    // reduced row echelon form with partial pivoting
    std::vector<int> pivot_col;
    int row = 0;
    for (int col = 0; col < n && row < m; ++col) {
        int best = row;
        for (int r = row + 1; r < m; ++r)
            if (fabs(L[r][col]) > fabs(L[best][col])) best = r;
        if (fabs(L[best][col]) < 1e-12) continue;
        std::swap(L[row], L[best]);
        const double p = L[row][col];
        for (int q = 0; q < n; ++q) L[row][q] /= p;
        for (int r = 0; r < m; ++r)
            if (r != row && L[r][col] != 0.0) {
                const double f = L[r][col];
                for (int q = 0; q < n; ++q) L[r][q] -= f * L[row][q];
            }
        pivot_col.push_back(col);
        ++row;
    }
    // one null vector per free column
    for (int col = 0; col < n; ++col) {
        bool is_pivot = false;
        for (int pc : pivot_col) is_pivot = is_pivot || pc == col;
        if (is_pivot) continue;
        std::vector<double> v(n, 0.0);
        v[col] = 1.0;
        for (size_t r = 0; r < pivot_col.size(); ++r) v[pivot_col[r]] = -L[r][col];
        basis.push_back(v);
    }
    return basis;
}

double factorial_d(int n) { double f = 1.0; for (int q = 2; q <= n; ++q) f *= q; return f; }

}  // namespace

// Q_0 .. Q_lmax concatenated row-major (host memory, Q_TOTAL doubles for l <= 5).
void build_q_tables(double *out) {
    for (int l = 0; l <= ANG_LMAX; ++l) {
        const std::vector<Exps> e = monomials(l);
        const int n = (int)e.size();
        std::vector<double> w(n);   // metric 1 / D_l
        for (int q = 0; q < n; ++q) w[q] = factorial_d(e[q].ax) * factorial_d(e[q].ay) * factorial_d(e[q].az) / factorial_d(l);
        std::vector<std::vector<double>> b = harmonic_basis(l);
        for (size_t r = 0; r < b.size(); ++r) {
            for (int pass = 0; pass < 2; ++pass)   // (second pass: re-orthogonalisation)
                for (size_t p = 0; p < r; ++p) {
                    double dot = 0.0;
                    for (int q = 0; q < n; ++q) dot += b[r][q] * b[p][q] * w[q];
                    for (int q = 0; q < n; ++q) b[r][q] -= dot * b[p][q];
                }
            double norm = 0.0;
            for (int q = 0; q < n; ++q) norm += b[r][q] * b[r][q] * w[q];
            norm = sqrt(norm);
            for (int q = 0; q < n; ++q) b[r][q] /= norm;
        }
        double *ql = out + q_offset(l);
        for (size_t r = 0; r < b.size(); ++r)
            for (int q = 0; q < n; ++q) ql[r * n + q] = b[r][q];
    }
}

}  // namespace mlip
