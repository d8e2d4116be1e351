/*
 * CPU fp64 oracle for the small-footprint MLIP hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against; nothing in the product path may call it, and
 * it shares no code, header, table or constant generator with the CUDA side.
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC (no fused multiply-add,
 * so the neighbor predicate rounds exactly as written).
 *
 * What is defined where (paper sections / equations):
 *   pair geometry                         Eq. 1        -> pair_geometry
 *   radial feature  g = E(r; s_i, s_j)    Eq. 2, Sec. 3.2.1 (pair-conditioned,
 *                                          C^2 networks), Sec. 4.1.3 (3 hidden
 *                                          layers of 128, SiLU, residual)
 *                                                      -> oracle_encoder, oracle_radial
 *   angular feature h = Omega_lmax(r^)    Eq. 3, Sec. 3.3.1 (Q_l applied to the
 *                                          degree-l monomials) -> oracle_angular
 *   moment P_i = sum_j h (x) g            Eq. 4        -> oracle_center
 *   invariants G_i                        Eq. 5 (C_l = I for the irreducible basis; the canonical monomial basis of
 *                                          Section 3.3, Eq. 11, with C_l = the multinomial multiplicities)
 *   energy E_i = R(G_i; s_i)              Eq. 6, Sec. 4.1.3 (4 hidden layers of
 *                                          64, SiLU, residual) -> oracle_head
 *   W_i, U_i, V_i                         Eq. 7-9
 *   partial force f_ij                    Eq. 10; forces are their scatter-sum
 *   neighbor set N(i)                     Sec. 3.1.1 ("within a given cutoff")
 *
 * Readings where the paper is silent (also listed in the design notes):
 *   - smooth cutoff: g is multiplied by f_c(r) = (1 + cos(pi r / r_c)) / 2;
 *   - residual connections wrap every hidden layer whose input and output
 *     widths agree (encoder layers 2.., head layers 2..); outputs are linear;
 *   - the encoder input is the bare distance in Angstrom;
 *   - virial Xi_ab = - sum_i sum_j (r_ij)_a (f_ij)_b  (the paper defines none);
 *   - minimum image by comparison with half the box edge; d^2 < r^2 is strict.
 *
 * Parity status: the paper prints no numeric energy or force, so the values of
 * E and F are pinned only through invariants and closed forms (finite
 * differences, three-body Legendre sums, dimer, l_max = 0 pair functional,
 * lattice shell counts, brute-force neighbor search); see tests/.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int n_species;    /* C */
    int k;            /* radial channels */
    int l_max;        /* angular order */
    int enc_hidden, enc_layers;
    int head_hidden, head_layers;
    double r_cut;
    const double *enc_w;   /* encoder nets, indexed by enc_net_index() */
    const double *head_w;  /* head nets, indexed by head_net_index() */
    const double *q;       /* Q_0 .. Q_lmax, row-major, concatenated */
    int chi_e;             /* species information given to the encoder (Section 3.2.2): 0 = pair (s_i, s_j), C*C nets;
                              1 = neighbor species s_j, C nets; 2 = none, one net */
    int chi_r;             /* ... to the regression network: 0 = central species s_i, C nets; 1 = none, one net */
    int envelope;          /* smooth cutoff (the paper names none): 0 = (1 + cos(pi x)) / 2, 1 = 1 - 10 x^3 + 15 x^4 - 6 x^5, x = r / r_c */
    int basis;             /* angular basis (Section 3.3): 0 = irreducible, block l has 2l+1 rows Q_l m_l(u), C_l = I;
                              1 = canonical, block l holds all C(l+2,2) monomials of degree l (q = identity blocks),
                              C_l = diag(l! / (ax! ay! az!)), the "Cartesian multiplicities" of Eq. 5 */
    const double *metric;  /* diagonal of C_0 .. C_lmax, one entry per row of the angular feature vector */
} oracle_model;

static int enc_net_index(const oracle_model *m, int si, int sj) {
    if (m->chi_e == 2) return 0;
    if (m->chi_e == 1) return sj;
    return si * m->n_species + sj;
}
static int head_net_index(const oracle_model *m, int si) { return m->chi_r == 1 ? 0 : si; }

static int n_mono(int l) { return (l + 1) * (l + 2) / 2; }
static int blk_rows(const oracle_model *m, int l) { return m->basis == 1 ? n_mono(l) : 2 * l + 1; }
static int ang_dim(const oracle_model *m) {
    int d = 0;
    for (int l = 0; l <= m->l_max; ++l) d += blk_rows(m, l);
    return d;
}

static double ipow(double x, int n) { double p = 1.0; for (int i = 0; i < n; ++i) p *= x; return p; }

static double sigmoid(double x) { return 1.0 / (1.0 + exp(-x)); }
static double silu(double x) { return x * sigmoid(x); }
static double dsilu(double x) { double s = sigmoid(x); return s * (1.0 + x * (1.0 - s)); }

static size_t enc_net_size(const oracle_model *m) {
    size_t h = (size_t)m->enc_hidden;
    return h + h + (size_t)(m->enc_layers - 1) * (h * h + h) + (size_t)m->k * h + (size_t)m->k;
}
static size_t head_net_size(const oracle_model *m) {
    size_t h = (size_t)m->head_hidden, n_in = (size_t)(m->l_max + 1) * (size_t)m->k;
    return n_in * h + h + (size_t)(m->head_layers - 1) * (h * h + h) + h + 1;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---- Eq. 3: h = [Q_0 m_0(u); Q_1 m_1(u); ...], and dh/du with u treated as free ---- */
void oracle_angular(const oracle_model *m, const double u[3], double *h, double *dh /* [d][3] */) {
    const double *q = m->q;
    int row0 = 0;
    for (int l = 0; l <= m->l_max; ++l) {
        int nm = n_mono(l);
        double mono[64], dmono[64][3];
        int col = 0;
        for (int ax = l; ax >= 0; --ax)
            for (int ay = l - ax; ay >= 0; --ay) {
                int az = l - ax - ay;
                mono[col] = ipow(u[0], ax) * ipow(u[1], ay) * ipow(u[2], az);
                dmono[col][0] = ax ? ax * ipow(u[0], ax - 1) * ipow(u[1], ay) * ipow(u[2], az) : 0.0;
                dmono[col][1] = ay ? ay * ipow(u[0], ax) * ipow(u[1], ay - 1) * ipow(u[2], az) : 0.0;
                dmono[col][2] = az ? az * ipow(u[0], ax) * ipow(u[1], ay) * ipow(u[2], az - 1) : 0.0;
                ++col;
            }
        for (int r = 0; r < blk_rows(m, l); ++r) {
            double s = 0.0, d0 = 0.0, d1 = 0.0, d2 = 0.0;
            for (int c = 0; c < nm; ++c) {
                double qrc = q[r * nm + c];
                s += qrc * mono[c];
                d0 += qrc * dmono[c][0];
                d1 += qrc * dmono[c][1];
                d2 += qrc * dmono[c][2];
            }
            h[row0 + r] = s;
            dh[(row0 + r) * 3 + 0] = d0;
            dh[(row0 + r) * 3 + 1] = d1;
            dh[(row0 + r) * 3 + 2] = d2;
        }
        q += blk_rows(m, l) * nm;
        row0 += blk_rows(m, l);
    }
}

/* ---- Eq. 2: encoder network of the ordered pair (s_i, s_j): y(r) and dy/dr ---- */
void oracle_encoder(const oracle_model *m, int si, int sj, double r, double *y, double *dy) {
    const int H = m->enc_hidden, K = m->k;
    const double *w = m->enc_w + (size_t)enc_net_index(m, si, sj) * enc_net_size(m);
    double a[H], da[H], pre[H], dpre[H];
    const double *W = w, *b = w + H;
    for (int o = 0; o < H; ++o) {
        double p = W[o] * r + b[o];
        a[o] = silu(p);
        da[o] = dsilu(p) * W[o];
    }
    w += 2 * H;
    for (int layer = 1; layer < m->enc_layers; ++layer) {
        W = w; b = w + (size_t)H * H;
        for (int o = 0; o < H; ++o) {
            double p = b[o], dp = 0.0;
            for (int i = 0; i < H; ++i) { p += W[o * H + i] * a[i]; dp += W[o * H + i] * da[i]; }
            pre[o] = p; dpre[o] = dp;
        }
        for (int o = 0; o < H; ++o) {      /* residual: a <- a + SiLU(W a + b) */
            a[o] += silu(pre[o]);
            da[o] += dsilu(pre[o]) * dpre[o];
        }
        w += (size_t)H * H + H;
    }
    W = w; b = w + (size_t)K * H;
    for (int c = 0; c < K; ++c) {
        double s = b[c], ds = 0.0;
        for (int i = 0; i < H; ++i) { s += W[c * H + i] * a[i]; ds += W[c * H + i] * da[i]; }
        y[c] = s; dy[c] = ds;
    }
}

/* smooth cutoff and its derivative: cosine, or the quintic that also has a vanishing second derivative at both ends */
static void envelope(int kind, double r, double r_cut, double *fc, double *dfc) {
    if (r >= r_cut) { *fc = 0.0; *dfc = 0.0; return; }
    if (kind == 1) {
        double x = r / r_cut;
        *fc = 1.0 - 10.0 * x * x * x + 15.0 * x * x * x * x - 6.0 * x * x * x * x * x;
        *dfc = (-30.0 * x * x + 60.0 * x * x * x - 30.0 * x * x * x * x) / r_cut;
    } else {
        double x = M_PI * r / r_cut;
        *fc = 0.5 * (1.0 + cos(x));
        *dfc = -0.5 * (M_PI / r_cut) * sin(x);
    }
}

/* radial feature g = f_c(r) E(r) and dg/dr */
void oracle_radial(const oracle_model *m, int si, int sj, double r, double *g, double *dg) {
    double y[m->k], dy[m->k], fc, dfc;
    oracle_encoder(m, si, sj, r, y, dy);
    envelope(m->envelope, r, m->r_cut, &fc, &dfc);
    for (int c = 0; c < m->k; ++c) { g[c] = fc * y[c]; dg[c] = dfc * y[c] + fc * dy[c]; }
}

/* ---- Eq. 6: head of species s: E = R(G); optionally dE/dG ---- */
double oracle_head(const oracle_model *m, int s, const double *G, double *dG /* may be NULL */) {
    const int H = m->head_hidden, L = m->head_layers, n_in = (m->l_max + 1) * m->k;
    const double *w0 = m->head_w + (size_t)head_net_index(m, s) * head_net_size(m);
    double pre[L][H], z[H];
    const double *w = w0;
    for (int o = 0; o < H; ++o) {
        double p = w[(size_t)n_in * H + o];
        for (int i = 0; i < n_in; ++i) p += w[(size_t)o * n_in + i] * G[i];
        pre[0][o] = p;
        z[o] = silu(p);
    }
    w += (size_t)n_in * H + H;
    for (int layer = 1; layer < L; ++layer) {
        for (int o = 0; o < H; ++o) {
            double p = w[(size_t)H * H + o];
            for (int i = 0; i < H; ++i) p += w[o * H + i] * z[i];
            pre[layer][o] = p;
        }
        for (int o = 0; o < H; ++o) z[o] += silu(pre[layer][o]);   /* residual */
        w += (size_t)H * H + H;
    }
    double e = w[H];
    for (int i = 0; i < H; ++i) e += w[i] * z[i];
    if (!dG) return e;

    /* reverse pass */
    double dz[H], dpre[H];
    for (int i = 0; i < H; ++i) dz[i] = w[i];
    for (int layer = L - 1; layer >= 1; --layer) {
        w -= (size_t)H * H + H;
        for (int o = 0; o < H; ++o) dpre[o] = dz[o] * dsilu(pre[layer][o]);
        for (int i = 0; i < H; ++i) {
            double s2 = 0.0;
            for (int o = 0; o < H; ++o) s2 += w[o * H + i] * dpre[o];
            dz[i] += s2;                                           /* skip path + layer path */
        }
    }
    w = w0;
    for (int o = 0; o < H; ++o) dpre[o] = dz[o] * dsilu(pre[0][o]);
    for (int i = 0; i < n_in; ++i) {
        double s2 = 0.0;
        for (int o = 0; o < H; ++o) s2 += w[(size_t)o * n_in + i] * dpre[o];
        dG[i] = s2;
    }
    return e;
}

/* ---- Eq. 1 with the periodic minimum image; returns d^2 ---- */
static double min_image(double d, double L) {
    double half = 0.5 * L;
    if (d > half) d -= L;
    else if (d < -half) d += L;
    return d;
}
static double pair_geometry(const double *pos, const double *box, int64_t i, int64_t j, double d[3]) {
    for (int a = 0; a < 3; ++a) d[a] = min_image(pos[3 * j + a] - pos[3 * i + a], box[a]);
    return (d[0] * d[0] + d[1] * d[1]) + d[2] * d[2];
}

/*
 * One central atom: Encoding (Eq. 1-5), Regression (Eq. 6), Derivation (Eq. 7-10).
 * list = the atom's neighbor list (any order), n_list entries, entries beyond r_cut
 * contribute nothing.  Outputs: E_i, optional G_i [(l_max+1)*k], optional partial
 * forces f_ij = dE_i/dr_ij [n_list][3] and their vectors r_ij [n_list][3].
 */
static double oracle_center(const oracle_model *m, int64_t i, const double *pos, const int32_t *species,
                            const double *box, const int32_t *list, int64_t n_list,
                            double *G_out, double *f_out, double *rij_out) {
    const int K = m->k, D = ang_dim(m), NG = (m->l_max + 1) * K;
    const int si = species[i];
    const double rc2 = m->r_cut * m->r_cut;
    double P[D][K], G[NG], dG[NG], W[D][K];
    double g[K], dg[K], h[D], dh[D][3];
    memset(P, 0, sizeof P);

    /* Encoding */
    for (int64_t n = 0; n < n_list; ++n) {
        double d[3], d2 = pair_geometry(pos, box, i, list[n], d);
        if (!(d2 < rc2)) continue;
        double r = sqrt(d2), u[3] = {d[0] / r, d[1] / r, d[2] / r};
        oracle_radial(m, si, species[list[n]], r, g, dg);
        oracle_angular(m, u, h, &dh[0][0]);
        for (int a = 0; a < D; ++a)
            for (int c = 0; c < K; ++c) P[a][c] += h[a] * g[c];          /* Eq. 4 */
    }
    for (int c = 0; c < K; ++c) G[c] = P[0][c];                           /* Eq. 5, l = 0 */
    for (int l = 1, row = 1; l <= m->l_max; row += blk_rows(m, l), ++l)
        for (int c = 0; c < K; ++c) {
            double s = 0.0;
            for (int a = row; a < row + blk_rows(m, l); ++a) s += m->metric[a] * P[a][c] * P[a][c];
            G[l * K + c] = s;                                             /* Eq. 5: p^T C_l p */
        }
    if (G_out) memcpy(G_out, G, sizeof G);

    /* Regression */
    double e = oracle_head(m, si, G, f_out ? dG : NULL);
    if (!f_out) return e;

    /* Derivation: W = dE/dP (Eq. 7) */
    for (int c = 0; c < K; ++c) W[0][c] = dG[c];
    for (int l = 1, row = 1; l <= m->l_max; row += blk_rows(m, l), ++l)
        for (int a = row; a < row + blk_rows(m, l); ++a)
            for (int c = 0; c < K; ++c) W[a][c] = 2.0 * dG[l * K + c] * m->metric[a] * P[a][c];

    for (int64_t n = 0; n < n_list; ++n) {
        double d[3], d2 = pair_geometry(pos, box, i, list[n], d);
        f_out[3 * n + 0] = f_out[3 * n + 1] = f_out[3 * n + 2] = 0.0;
        rij_out[3 * n + 0] = d[0]; rij_out[3 * n + 1] = d[1]; rij_out[3 * n + 2] = d[2];
        if (!(d2 < rc2)) continue;
        double r = sqrt(d2), u[3] = {d[0] / r, d[1] / r, d[2] / r};
        oracle_radial(m, si, species[list[n]], r, g, dg);
        oracle_angular(m, u, h, &dh[0][0]);
        double urow[K], vrow[D];
        for (int c = 0; c < K; ++c) {                                     /* Eq. 8: row of U = G_ang W */
            double s = 0.0;
            for (int a = 0; a < D; ++a) s += h[a] * W[a][c];
            urow[c] = s;
        }
        for (int a = 0; a < D; ++a) {                                     /* Eq. 9: row of V = G_rad W^T */
            double s = 0.0;
            for (int c = 0; c < K; ++c) s += g[c] * W[a][c];
            vrow[a] = s;
        }
        /* Eq. 10.  J_rad = dg/dr_ij = g'(r) (x) r^ ;  J_ang = (dh/du)(I - u u^T)/r */
        double s_rad = 0.0;
        for (int c = 0; c < K; ++c) s_rad += dg[c] * urow[c];
        double t[3] = {0.0, 0.0, 0.0};
        for (int a = 0; a < D; ++a)
            for (int b = 0; b < 3; ++b) t[b] += vrow[a] * dh[a][b];
        double tu = t[0] * u[0] + t[1] * u[1] + t[2] * u[2];
        for (int b = 0; b < 3; ++b) f_out[3 * n + b] = s_rad * u[b] + (t[b] - tu * u[b]) / r;
    }
    return e;
}

/*
 * Energies, forces and virial from a set of central atoms.
 *   rows[q] (or q itself when rows == NULL) is the central atom of list row q;
 *   seg_ptr [n_rows*C + 1] and nbr hold species-segmented lists of those rows.
 *   e_atom [n_atoms]: written at the central atoms only.
 *   forces [n_atoms][3]: F_a = sum_j f_aj - sum_i f_ia accumulated over the given
 *   central atoms only (the full force when every atom is a central atom).
 *   virial [9] row-major, energy = sum of the central atoms' E_i.
 */
int oracle_compute(const oracle_model *m, int64_t n_atoms, const double *pos, const int32_t *species,
                   const double *box, int64_t n_rows, const int64_t *rows, const int64_t *seg_ptr,
                   const int32_t *nbr, double *e_atom, double *forces, double *virial, double *energy,
                   double *G_out) {
    const int C = m->n_species, NG = (m->l_max + 1) * m->k;
    double e_tot = 0.0, vir[9] = {0};
    memset(forces, 0, sizeof(double) * 3 * (size_t)n_atoms);
#pragma omp parallel
    {
        double e_loc = 0.0, v_loc[9] = {0};
        double *f = NULL, *rij = NULL;
        int64_t cap = 0;
#pragma omp for schedule(dynamic, 8)
        for (int64_t q = 0; q < n_rows; ++q) {
            int64_t i = rows ? rows[q] : q;
            int64_t beg = seg_ptr[q * C], n_list = seg_ptr[(q + 1) * C] - beg;
            if (n_list > cap) {
                cap = n_list + 64;
                f = realloc(f, sizeof(double) * 3 * cap);
                rij = realloc(rij, sizeof(double) * 3 * cap);
            }
            double e = oracle_center(m, i, pos, species, box, nbr + beg, n_list,
                                     G_out ? G_out + (size_t)q * NG : NULL, f, rij);
            e_atom[i] = e;
            e_loc += e;
            double fi[3] = {0, 0, 0};
            for (int64_t n = 0; n < n_list; ++n) {
                int64_t j = nbr[beg + n];
                for (int b = 0; b < 3; ++b) {
                    fi[b] += f[3 * n + b];
#pragma omp atomic
                    forces[3 * j + b] -= f[3 * n + b];
                    for (int a = 0; a < 3; ++a) v_loc[3 * a + b] -= rij[3 * n + a] * f[3 * n + b];
                }
            }
            for (int b = 0; b < 3; ++b) {
#pragma omp atomic
                forces[3 * i + b] += fi[b];
            }
        }
        free(f); free(rij);
#pragma omp critical
        {
            e_tot += e_loc;
            for (int a = 0; a < 9; ++a) vir[a] += v_loc[a];
        }
    }
    *energy = e_tot;
    memcpy(virial, vir, sizeof vir);
    return 0;
}

/* ---------------- neighbor lists ---------------- */

/*
 * Brute force over all atoms.  Row q lists, for s = 0..C-1, every j != i of
 * species s with minimum-image d^2 < r_list^2, ascending j.  Returns the total
 * number of entries; nbr is only written while it fits in cap.
 */
int64_t oracle_neighbors_brute(int64_t n, const double *pos, const int32_t *species, int C,
                               const double *box, double r_list, int64_t n_rows, const int64_t *rows,
                               int64_t *seg_ptr, int32_t *nbr, int64_t cap) {
    const double rl2 = r_list * r_list;
    int64_t total = 0;
    for (int64_t q = 0; q < n_rows; ++q) {
        int64_t i = rows ? rows[q] : q;
        for (int s = 0; s < C; ++s) {
            seg_ptr[q * C + s] = total;
            for (int64_t j = 0; j < n; ++j) {
                if (j == i || species[j] != s) continue;
                double d[3];
                if (pair_geometry(pos, box, i, j, d) < rl2) {
                    if (total < cap) nbr[total] = (int32_t)j;
                    ++total;
                }
            }
        }
    }
    seg_ptr[n_rows * C] = total;
    return total;
}

static int cmp_i64(const void *a, const void *b) {
    int64_t x = *(const int64_t *)a, y = *(const int64_t *)b;
    return (x > y) - (x < y);
}

/* Same lists through a cell grid (cells no smaller than r_list), for large n. */
int64_t oracle_neighbors_cell(int64_t n, const double *pos, const int32_t *species, int C,
                              const double *box, double r_list, int64_t n_rows, const int64_t *rows,
                              int64_t *seg_ptr, int32_t *nbr, int64_t cap) {
    const double rl2 = r_list * r_list;
    int nc[3];
    double edge[3];
    for (int a = 0; a < 3; ++a) {
        nc[a] = (int)floor(box[a] / r_list);
        if (nc[a] < 1) nc[a] = 1;
        edge[a] = box[a] / nc[a];
    }
    int64_t n_cells = (int64_t)nc[0] * nc[1] * nc[2];
    int64_t *cell_start = calloc((size_t)n_cells + 1, sizeof(int64_t));
    int64_t *cell_of = malloc(sizeof(int64_t) * (size_t)n);
    int32_t *cell_atoms = malloc(sizeof(int32_t) * (size_t)n);
    for (int64_t i = 0; i < n; ++i) {
        int c[3];
        for (int a = 0; a < 3; ++a) {
            c[a] = (int)floor(pos[3 * i + a] / edge[a]);
            if (c[a] < 0) c[a] = 0;
            if (c[a] >= nc[a]) c[a] = nc[a] - 1;
        }
        cell_of[i] = ((int64_t)c[0] * nc[1] + c[1]) * nc[2] + c[2];
        cell_start[cell_of[i] + 1]++;
    }
    for (int64_t c = 0; c < n_cells; ++c) cell_start[c + 1] += cell_start[c];
    int64_t *fill = malloc(sizeof(int64_t) * (size_t)n_cells);
    memcpy(fill, cell_start, sizeof(int64_t) * (size_t)n_cells);
    for (int64_t i = 0; i < n; ++i) cell_atoms[fill[cell_of[i]]++] = (int32_t)i;
    free(fill);

    int64_t *count = calloc((size_t)n_rows + 1, sizeof(int64_t));
    for (int pass = 0; pass < 2; ++pass) {
#pragma omp parallel
        {
            int64_t *keys = NULL, kcap = 0;
#pragma omp for schedule(dynamic, 64)
            for (int64_t q = 0; q < n_rows; ++q) {
                int64_t i = rows ? rows[q] : q, nk = 0;
                int64_t ci = cell_of[i];
                int c0[3] = {(int)(ci / ((int64_t)nc[1] * nc[2])), (int)((ci / nc[2]) % nc[1]), (int)(ci % nc[2])};
                int lst[3][3], nl[3];
                for (int a = 0; a < 3; ++a) {      /* distinct cells c-1, c, c+1 (periodic) */
                    nl[a] = 0;
                    for (int o = -1; o <= 1; ++o) {
                        int c = ((c0[a] + o) % nc[a] + nc[a]) % nc[a], dup = 0;
                        for (int t = 0; t < nl[a]; ++t) dup |= (lst[a][t] == c);
                        if (!dup) lst[a][nl[a]++] = c;
                    }
                }
                for (int x = 0; x < nl[0]; ++x)
                    for (int y = 0; y < nl[1]; ++y)
                        for (int z = 0; z < nl[2]; ++z) {
                            int64_t c = ((int64_t)lst[0][x] * nc[1] + lst[1][y]) * nc[2] + lst[2][z];
                            for (int64_t p = cell_start[c]; p < cell_start[c + 1]; ++p) {
                                int64_t j = cell_atoms[p];
                                double d[3];
                                if (j == i || !(pair_geometry(pos, box, i, j, d) < rl2)) continue;
                                if (nk == kcap) { kcap = 2 * kcap + 64; keys = realloc(keys, sizeof(int64_t) * kcap); }
                                keys[nk++] = ((int64_t)species[j] << 32) | j;
                            }
                        }
                if (pass == 0) { count[q + 1] = nk; continue; }
                qsort(keys, (size_t)nk, sizeof(int64_t), cmp_i64);
                int64_t beg = count[q];
                int s = 0;
                seg_ptr[q * C] = beg;
                for (int64_t t = 0; t < nk; ++t) {
                    int sj = (int)(keys[t] >> 32);
                    while (s < sj) seg_ptr[q * C + (++s)] = beg + t;
                    if (beg + t < cap) nbr[beg + t] = (int32_t)(keys[t] & 0xffffffff);
                }
                while (s < C - 1) seg_ptr[q * C + (++s)] = beg + nk;
            }
            free(keys);
        }
        if (pass == 0)
            for (int64_t q = 0; q < n_rows; ++q) count[q + 1] += count[q];
    }
    int64_t total = count[n_rows];
    seg_ptr[n_rows * C] = total;
    free(count); free(cell_start); free(cell_of); free(cell_atoms);
    return total;
}
