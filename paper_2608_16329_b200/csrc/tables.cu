// Radial tables.  The radial feature of Eq. 2, g(r) = f_c(r) E(r; s_i, s_j), is a function of
// one scalar per ordered species pair, so each encoder network (Section 4.1.3: three hidden
// layers of width 128, SiLU, residual) is evaluated once per knot here, in fp64, and replaced
// by a C^2 cubic B-spline with clamped (first-derivative) ends on [r_min, r_cut].  g'(r) used
// by the force (Eq. 10) is the exact derivative of that spline, so energies and forces stay
// consistent.  The spline is then compared with the network between the knots.
#include "common.cuh"

namespace mlip {

constexpr int MAX_ENC_H = 256;

struct EncShape { int hidden, layers, k, n_species; double r_cut; int envelope; };

__device__ inline double d_sigmoid(double x) { return 1.0 / (1.0 + exp(-x)); }

// Encoder value and derivative (forward mode) times the smooth cutoff.
__device__ void eval_radial(const double *__restrict__ w, EncShape sh, double r, double *g, double *dg) {
    const int H = sh.hidden;
    double a[MAX_ENC_H], da[MAX_ENC_H], pre[MAX_ENC_H], dpre[MAX_ENC_H];
    for (int o = 0; o < H; ++o) {
        double p = w[o] * r + w[H + o], s = d_sigmoid(p);
        a[o] = p * s;
        da[o] = s * (1.0 + p * (1.0 - s)) * w[o];
    }
    w += 2 * H;
    for (int layer = 1; layer < sh.layers; ++layer) {
        const double *b = w + (size_t)H * H;
        for (int o = 0; o < H; ++o) {
            double p = b[o], dp = 0.0;
            const double *row = w + (size_t)o * H;
            for (int i = 0; i < H; ++i) { p += row[i] * a[i]; dp += row[i] * da[i]; }
            pre[o] = p; dpre[o] = dp;
        }
        for (int o = 0; o < H; ++o) {
            double p = pre[o], s = d_sigmoid(p);
            a[o] += p * s;
            da[o] += s * (1.0 + p * (1.0 - s)) * dpre[o];
        }
        w += (size_t)H * H + H;
    }
    double fc = 0.0, dfc = 0.0;   // smooth cutoff: cosine or quintic polynomial
    if (r < sh.r_cut) {
        if (sh.envelope == 1) {
            const double x = r / sh.r_cut, x2 = x * x;
            fc = 1.0 + x2 * x * (-10.0 + x * (15.0 - 6.0 * x));
            dfc = x2 * (-30.0 + x * (60.0 - 30.0 * x)) / sh.r_cut;
        } else {
            const double x = M_PI * r / sh.r_cut;
            fc = 0.5 * (1.0 + cos(x));
            dfc = -0.5 * (M_PI / sh.r_cut) * sin(x);
        }
    }
    const double *b = w + (size_t)sh.k * H;
    for (int c = 0; c < sh.k; ++c) {
        double y = b[c], dy = 0.0;
        const double *row = w + (size_t)c * H;
        for (int i = 0; i < H; ++i) { y += row[i] * a[i]; dy += row[i] * da[i]; }
        g[c] = fc * y;
        dg[c] = dfc * y + fc * dy;
    }
}

// samples: [net][point][k] values and derivatives at r = r0 + point * step
__global__ void k_table_sample(const double *__restrict__ enc_w, size_t net_size, EncShape sh, int n_nets, int n_points,
                               double r0, double step, double r_last, double *__restrict__ val, double *__restrict__ der) {
    int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_nets * n_points) return;
    int net = t / n_points, p = t % n_points;
    double r = p == n_points - 1 ? r_last : r0 + p * step;
    double g[MAX_K], dg[MAX_K];
    eval_radial(enc_w + (size_t)net * net_size, sh, r, g, dg);
    for (int c = 0; c < sh.k; ++c) {
        val[((size_t)net * n_points + p) * sh.k + c] = g[c];
        der[((size_t)net * n_points + p) * sh.k + c] = dg[c];
    }
}

// One thread per (net, channel): clamped cubic B-spline interpolation through the K + 1 knot values.
// Unknown control points c_0 .. c_{K+2};  (c_i + 4 c_{i+1} + c_{i+2}) / 6 = f_i,  (c_2 - c_0) / 2h = f'_0,
// (c_{K+2} - c_K) / 2h = f'_K.  Thomas algorithm on c_1 .. c_{K+1}; `work` holds 2 (K + 1) doubles per thread.
template <typename CoefT>
__global__ void k_table_solve(const double *__restrict__ val, const double *__restrict__ der, int n_nets, int knots, int k,
                              double h, double *__restrict__ work, CoefT *__restrict__ coef) {
    int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_nets * k) return;
    const int net = t / k, c = t % k, n = knots + 1;
    const double *f = val + (size_t)net * n * k + c, *fp = der + (size_t)net * n * k + c;
    double *cp = work + (size_t)t * 2 * n, *x = cp + n;
    // row 0: 4 c1 + 2 c2 = 6 f0 + 2 h f'0 ; rows i: c_i + 4 c_{i+1} + c_{i+2} = 6 f_i ; last: 2 c_K + 4 c_{K+1} = 6 f_K - 2 h f'_K
    double diag = 4.0, upper = 2.0, rhs = 6.0 * f[0] + 2.0 * h * fp[0];
    cp[0] = upper / diag;
    x[0] = rhs / diag;
    for (int i = 1; i < n; ++i) {
        double lower = (i == n - 1) ? 2.0 : 1.0;
        upper = 1.0;
        rhs = (i == n - 1) ? 6.0 * f[(size_t)i * k] - 2.0 * h * fp[(size_t)i * k] : 6.0 * f[(size_t)i * k];
        double m = 4.0 - lower * cp[i - 1];
        cp[i] = upper / m;
        x[i] = (rhs - lower * x[i - 1]) / m;
    }
    for (int i = n - 2; i >= 0; --i) x[i] -= cp[i] * x[i + 1];
    CoefT *out = coef + (size_t)net * (knots + 3) * k + c;
    out[0] = (CoefT)(x[1] - 2.0 * h * fp[0]);                        // c_0 = c_2 - 2 h f'_0
    for (int i = 0; i < n; ++i) out[(size_t)(i + 1) * k] = (CoefT)x[i];
    out[(size_t)(knots + 2) * k] = (CoefT)(x[n - 2] + 2.0 * h * fp[(size_t)(n - 1) * k]);
}

__device__ inline void atomic_max_pos(unsigned long long *addr, double v) {   // v >= 0: bit patterns are ordered
    atomicMax(addr, (unsigned long long)__double_as_longlong(v));
}

// Compare the stored spline (evaluated in fp64) with network samples taken between the knots.
// out[0] = max |g|, out[1] = max |g'|, out[2] = max |spline - g|, out[3] = max |spline' - g'|
template <typename CoefT>
__global__ void k_table_check(const double *__restrict__ val, const double *__restrict__ der, const CoefT *__restrict__ coef,
                              int n_nets, int n_points, int knots, int k, double r_min, double r0, double step, double h,
                              unsigned long long *out) {
    int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_nets * n_points) return;
    int net = t / n_points, p = t % n_points;
    double r = r0 + p * step;
    double xk = (r - r_min) / h;
    int i = (int)floor(xk);
    i = i < 0 ? 0 : (i > knots - 1 ? knots - 1 : i);
    double u = xk - i, u2 = u * u, u3 = u2 * u, v = 1.0 - u;
    double b[4] = {v * v * v / 6.0, (3.0 * u3 - 6.0 * u2 + 4.0) / 6.0, (-3.0 * u3 + 3.0 * u2 + 3.0 * u + 1.0) / 6.0, u3 / 6.0};
    double db[4] = {-0.5 * v * v / h, (1.5 * u2 - 2.0 * u) / h, (-1.5 * u2 + u + 0.5) / h, 0.5 * u2 / h};
    double m[4] = {0, 0, 0, 0};
    for (int c = 0; c < k; ++c) {
        const CoefT *cf = coef + ((size_t)net * (knots + 3) + i) * k + c;
        double s = 0.0, ds = 0.0;
        for (int q = 0; q < 4; ++q) { s += b[q] * (double)cf[(size_t)q * k]; ds += db[q] * (double)cf[(size_t)q * k]; }
        double g = val[((size_t)net * n_points + p) * k + c], dg = der[((size_t)net * n_points + p) * k + c];
        m[0] = fmax(m[0], fabs(g)); m[1] = fmax(m[1], fabs(dg));
        m[2] = fmax(m[2], fabs(s - g)); m[3] = fmax(m[3], fabs(ds - dg));
    }
    for (int q = 0; q < 4; ++q) atomic_max_pos(out + q, m[q]);
}

int build_tables(mlip_ctx *c, const double *enc_w_host, size_t n_enc) {
    const mlip_config &cfg = c->cfg;
    const int C = cfg.n_species, n_nets = C * C, K = cfg.table_knots, k = cfg.k, H = cfg.enc_hidden;
    const size_t net_size = (size_t)H + H + (size_t)(cfg.enc_layers - 1) * ((size_t)H * H + H) + (size_t)k * H + k;
    if (n_enc != net_size * n_nets) { c->err = "encoder weight count does not match the configured shape"; return MLIP_ERR_INVALID_ARG; }
    if (H > MAX_ENC_H) { c->err = "enc_hidden above 256 is not compiled in"; return MLIP_ERR_UNSUPPORTED; }
    const double r_min = cfg.table_r_min, h = (cfg.r_cut - r_min) / K;
    const EncShape sh{H, cfg.enc_layers, k, C, cfg.r_cut, cfg.envelope};
    const int n_knot_pts = K + 1, n_chk = 4 * K;     // check at 4 points per interval, offset from the knots
    double *w = nullptr, *val = nullptr, *der = nullptr, *work = nullptr;
    unsigned long long *stats = nullptr;
    const size_t n_pts_max = (size_t)n_nets * n_chk * k;
    MLIP_CUDA_TRY(c, cudaMalloc(&w, sizeof(double) * n_enc));
    MLIP_CUDA_TRY(c, cudaMalloc(&val, sizeof(double) * n_pts_max));
    MLIP_CUDA_TRY(c, cudaMalloc(&der, sizeof(double) * n_pts_max));
    MLIP_CUDA_TRY(c, cudaMalloc(&work, sizeof(double) * (size_t)n_nets * k * 2 * n_knot_pts));
    MLIP_CUDA_TRY(c, cudaMalloc(&stats, sizeof(unsigned long long) * 4));
    const bool f64 = cfg.precision == 1;
    const size_t coef_bytes = (f64 ? sizeof(double) : sizeof(float)) * (size_t)n_nets * (K + 3) * k;
    if (c->table || c->table_d) {   // a retry with more knots
        cudaFree(c->table); cudaFree(c->table_d);
        c->table = nullptr; c->table_d = nullptr;
        c->resident -= c->table_bytes;
    }
    if (f64) MLIP_CUDA_TRY(c, cudaMalloc(&c->table_d, coef_bytes));
    else MLIP_CUDA_TRY(c, cudaMalloc(&c->table, coef_bytes));
    c->table_bytes = coef_bytes;
    c->resident += coef_bytes;
    c->kernel_ready = false;
    MLIP_CUDA_TRY(c, cudaMemcpy(w, enc_w_host, sizeof(double) * n_enc, cudaMemcpyHostToDevice));
    MLIP_CUDA_TRY(c, cudaMemset(stats, 0, sizeof(unsigned long long) * 4));

    int nt = n_nets * n_knot_pts;
    k_table_sample<<<(nt + 63) / 64, 64>>>(w, net_size, sh, n_nets, n_knot_pts, r_min, h, cfg.r_cut, val, der);
    if (f64) k_table_solve<double><<<(n_nets * k + 63) / 64, 64>>>(val, der, n_nets, K, k, h, work, c->table_d);
    else k_table_solve<float><<<(n_nets * k + 63) / 64, 64>>>(val, der, n_nets, K, k, h, work, c->table);
    nt = n_nets * n_chk;
    const double step = h / 4.0, r0 = r_min + 0.37 * step;
    k_table_sample<<<(nt + 63) / 64, 64>>>(w, net_size, sh, n_nets, n_chk, r0, step, r0 + (n_chk - 1) * step, val, der);
    if (f64) k_table_check<double><<<(nt + 63) / 64, 64>>>(val, der, c->table_d, n_nets, n_chk, K, k, r_min, r0, step, h, stats);
    else k_table_check<float><<<(nt + 63) / 64, 64>>>(val, der, c->table, n_nets, n_chk, K, k, r_min, r0, step, h, stats);
    c->launches += 4;
    unsigned long long host_stats[4];
    MLIP_CUDA_TRY(c, cudaMemcpy(host_stats, stats, sizeof host_stats, cudaMemcpyDeviceToHost));
    MLIP_CUDA_TRY(c, cudaDeviceSynchronize());
    cudaFree(w); cudaFree(val); cudaFree(der); cudaFree(work); cudaFree(stats);
    double m[4];
    for (int q = 0; q < 4; ++q) memcpy(&m[q], &host_stats[q], sizeof(double));
    c->table_err_value = m[0] > 0 ? m[2] / m[0] : 0.0;
    c->table_err_deriv = m[1] > 0 ? m[3] / m[1] : 0.0;
    c->tab.coef = c->table;
    c->tab.knots = K;
    c->tab.r_min = (float)r_min;
    c->tab.inv_h = (float)(1.0 / h);
    c->tab.r_cut2 = (float)(cfg.r_cut * cfg.r_cut);
    // the fp64 path also bounds the derivative (it carries the forces): one order in h worse than the value
    const bool value_ok = c->table_err_value <= cfg.table_tol;
    const bool deriv_ok = !f64 || c->table_err_deriv <= 100.0 * cfg.table_tol;
    if (!value_ok || !deriv_ok) {
        char buf[200];
        snprintf(buf, sizeof buf, "radial table error %.3g (derivative %.3g) exceeds table_tol %.3g; raise table_knots",
                 c->table_err_value, c->table_err_deriv, cfg.table_tol);
        c->err = buf;
        return MLIP_ERR_TABLE_TOLERANCE;
    }
    return MLIP_OK;
}

}  // namespace mlip
