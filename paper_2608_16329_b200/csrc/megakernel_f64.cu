// Double-precision evaluation path (`precision = 1`): the same fused pass as megakernel.cu --
// encoding (Eq. 1-5), regression (Eq. 6) and derivation (Eq. 7-10) of an atom back to back with
// nothing per pair or per atom written to device memory except forces and E_i -- in fp64.
// Section 4.2 evaluates the potential in double precision by default; this path is for validation
// and for runs that want that accuracy.
//
//   CTA = 8 warps = a tile of 8 atoms of one central species (atoms in (species, cell) order)
//   encoding    one warp per atom: lane = list entry for geometry, angular values and spline basis; then the
//               moment P = H^T G (Eq. 4) on the fp64 tensor pipe (mma.sync m8n8k4, IEEE fp64 FMA chains), four
//               pairs per step, with g (Eq. 2) evaluated straight into the B operand
//   regression  the whole CTA on the tile: every layer is W [64 x in] times the tile's activations
//               [in x 8 atoms] on the fp64 tensor pipe, warp = 8 rows of W, so each weight is read from L2 once
//               per tile instead of once per atom; the reverse pass reads transposed copies the same way
//   derivation  one warp per atom: [V; T] = [G; G'] W^T (Eq. 9 and the re-associated Eq. 8 term) on the tensor
//               pipe, eight pairs per tile, then lane = pair for the projection onto the pair vector and fp64
//               atomics for f_j
//
// What bounds this kernel is the L1 / shared-memory data pipe and L2 latency, not fp64 arithmetic: every global
// load is therefore shaped so that a quad or an eight-lane group reads 128 or 256 contiguous bytes (the k-index <->
// channel assignment of a contraction is free), and the staging rows in shared memory are padded against bank
// conflicts.
//
// The radial tables are the same clamped cubic B-splines as in the fp32 path but with fp64
// coefficients and enough knots for ~1e-11 relative error; they stay in global memory (L2).
//
// The kernel is a template over the descriptor shape: k in {16, 32, 64} radial channels,
// l_max in {1, 2, 3} (d = 4, 9, 16) with closed-form harmonics, plus (angular.cuh) l_max = 4, 5
// (d = 25, 36) through projection matrices and the canonical monomial basis (d = 4, 10, 20) with
// the metric C_l of Eq. 5 -- the throughput side of the paper's ablations (Tables 6, 7 and
// Fig. 4(c)).  With k = 16 the upper half-warp idles in the lane = channel phases; with k = 64
// a lane owns channels lane and lane + 32.
#include <algorithm>
#include <type_traits>

#include "angular.cuh"
#include "common.cuh"
#include "pair_math.cuh"

namespace mlip {

constexpr int F64_QCAP = 128;       // pairs per atom kept between the phases (more: the derivation scans the list again)
constexpr int F64_TILE = 8;         // atoms per tile = warps per CTA = columns of the tensor-pipe tile
constexpr int F64_YS = HEAD_H + 2;  // activation row stride: 2 mod 4 doubles keeps the 16-byte B-operand reads conflict-free

// per-species head block (doubles) for n_inv inputs: the caller's row-major matrices, then biases and output layer
struct Head64 {
    int w0, wl, w0t, wlt, bias, wout, total;
    __host__ __device__ constexpr explicit Head64(int n_inv)
        : w0(0),                                            // [64][n_inv]
          wl(HEAD_H * n_inv),                               // 3 x [64][64]
          w0t(wl + (HEAD_L - 1) * HEAD_H * HEAD_H),         // [n_inv][64]: the transposes feed the reverse pass rows too
          wlt(w0t + HEAD_H * n_inv),                        // 3 x [64][64]
          bias(wlt + (HEAD_L - 1) * HEAD_H * HEAD_H),       // [4][64]
          wout(bias + HEAD_L * HEAD_H),                     // [64] + b_out
          total(wout + HEAD_H + 8) {}
};

template <int K, int LMAX, int BASIS>
struct TileSmem {
    using Shape = AngShape<LMAX, BASIS>;
    static constexpr int D = Shape::D;
    static constexpr int NINV = (LMAX + 1) * K;
    static constexpr int XS = (NINV + 31) / 32 * 32 + 2;
    double x[F64_TILE][XS];                 // invariants, then dE/dG
    double y[2][F64_TILE][F64_YS];          // activations of the previous / current layer
    double sd[HEAD_L][F64_TILE][F64_YS];    // SiLU'(pre-activation) per layer
    double dp[2][F64_TILE][F64_YS];         // dE/dpre of the layer being propagated
    union {
        double dv[16 * (12 + 16 * ((D + 7) / 8))];   // derivation staging of the tensor form: 16 pairs x (b, b', offset | V, T, pad)
        double w[D * K];                    // W_i = dE_i/dP_i (Eq. 7), derivation; P_i on its way from fragments to lane = channel
        double te[(D + 5) * 36];            // encoding hand-over of the tensor form: D rows of h, 4 of b, table offsets, 32 pairs (+ 4 pad) each
    } pw[F64_TILE];
    int q[F64_TILE][F64_QCAP];              // neighbor indices of the pairs inside r_cut: kept from the encoding to the derivation
};

struct F64Args {
    int64_t n;
    int n_species;
    CellGrid grid;
    double rc2;
    const double *coef;
    int knots;
    double r_min, inv_h;
    const double4 *pos4;
    const int32_t *center_order;
    const int32_t *species_start;
    const int64_t *nbr_off;
    const int32_t *nbr_near;   // leading entries of each list that can be inside r_cut while far_flag is down
    const int *far_flag;
    const int32_t *nbr;
    const uint16_t *nbr16;     // non-null: the lists hold 16-bit cell-relative codes (decoded with cell_id / cell_start)
    const int32_t *cell_id, *cell_start;
    int64_t nbr_cap;           // entries the list array holds (range-checked builds)
    const double *head;
    double *force;      // [N][3]
    double *e_atom;
    double *acc;
    unsigned long long *pair_counter;
    int *status;
};

__device__ __forceinline__ double silu_d(double x, double &dsilu) {
    const double s = 1.0 / (1.0 + exp(-x));
    dsilu = s * (1.0 + x * (1.0 - s));
    return x * s;
}

// C[8 x 8] += A[8 x 4] B[4 x 8] in fp64: lane (g = lane / 4, t = lane % 4) holds A[g][t], B[t][g], C[g][2t], C[g][2t + 1]
__device__ __forceinline__ void dmma(double &c0, double &c1, double a, double b) {
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};" : "+d"(c0), "+d"(c1) : "d"(a), "d"(b));
}

// One row block of a head layer on the tensor pipe: c += A[8 x 16 NH] B[16 NH x 8].  The k-index <-> input assignment
// is free as long as both operands use it: k-step 4 h + u contracts input 16 h + 4 t + u, so a quad reads 128
// contiguous bytes of its weight row per load and a lane's four activations are two 16-byte shared-memory reads.
// wrow = the lane's weight row + 4 t, xrow = the activations of atom g + 4 t.  Two accumulator chains.
template <int NH>
__device__ __forceinline__ void head_dot(double &c0, double &c1, const double *__restrict__ wrow, const double *xrow) {
    double w[NH][4];
#pragma unroll
    for (int h = 0; h < NH; ++h)
        asm volatile("ld.global.nc.v4.f64 {%0,%1,%2,%3}, [%4];" : "=d"(w[h][0]), "=d"(w[h][1]), "=d"(w[h][2]), "=d"(w[h][3]) : "l"(wrow + 16 * h));
    double a0 = 0.0, a1 = 0.0;
#pragma unroll
    for (int h = 0; h < NH; ++h) {
        const double2 x01 = *reinterpret_cast<const double2 *>(xrow + 16 * h), x23 = *reinterpret_cast<const double2 *>(xrow + 16 * h + 2);
        if (h & 1) {
            dmma(a0, a1, w[h][0], x01.x); dmma(a0, a1, w[h][1], x01.y); dmma(a0, a1, w[h][2], x23.x); dmma(a0, a1, w[h][3], x23.y);
        } else {
            dmma(c0, c1, w[h][0], x01.x); dmma(c0, c1, w[h][1], x01.y); dmma(c0, c1, w[h][2], x23.x); dmma(c0, c1, w[h][3], x23.y);
        }
    }
    c0 += a0; c1 += a1;
}

#ifndef MLIP_F64_TWO_PER_SM_MAX_D
#define MLIP_F64_TWO_PER_SM_MAX_D 20
#endif
template <int K, int LMAX, int BASIS>
constexpr int f64_ctas_per_sm() { return (K <= 32 && AngShape<LMAX, BASIS>::D <= MLIP_F64_TWO_PER_SM_MAX_D) ? 2 : 1; }

template <int K, int LMAX, int BASIS>
__global__ void __launch_bounds__(F64_TILE * 32, f64_ctas_per_sm<K, LMAX, BASIS>()) k_mega_f64(F64Args k) {
    using SM = TileSmem<K, LMAX, BASIS>;
    using Shape = AngShape<LMAX, BASIS>;
    constexpr int D = SM::D, NINV = SM::NINV;
    constexpr bool CLOSED = BASIS == 0 && LMAX <= 3;   // the default basis up to l = 3 has hand-written harmonics
    constexpr int CPL = (K + 31) / 32;   // channels per lane
    constexpr Head64 H(NINV);
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SM &sm = *reinterpret_cast<SM *>(smem_raw);
    __shared__ int s_start[MAX_SPECIES + 1];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int C = k.n_species;
    // lists that an in-step rebuild could not complete (capacity, broken configuration) are not evaluated: the outputs
    // stay at their cleared values and the status word tells the caller why
    if (*k.status & (FLAG_NEIGHBOR_OVERFLOW | FLAG_NONFINITE)) return;
    const bool use_far = *k.far_flag != 0;   // an atom has moved skin / 4 since the build: every list entry counts
    if (threadIdx.x <= C) s_start[threadIdx.x] = k.species_start[threadIdx.x];
    __syncthreads();
    int total_tiles = 0;
    for (int s = 0; s < C; ++s) total_tiles += (s_start[s + 1] - s_start[s] + F64_TILE - 1) / F64_TILE;
    double e_sum = 0.0, vir[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};
    unsigned long long n_pairs = 0;
    PhaseClock pc;
    pc.start();

    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        int si = 0, tl = tile;
        for (;;) {   // tiles are numbered species by species
            const int nt = (s_start[si + 1] - s_start[si] + F64_TILE - 1) / F64_TILE;
            if (tl < nt) break;
            tl -= nt; ++si;
        }
        const int slot = s_start[si] + F64_TILE * tl + wid;
        const bool have = slot < s_start[si + 1];
        const double *hd = k.head + (size_t)si * H.total;
        int i = 0;
        double4 pi = make_double4(0.0, 0.0, 0.0, 0.0);
        int64_t beg = 0, end = 0;
        if (have) {
            i = (int)MLIP_CHECK_INDEX(k.center_order[slot], k.n, k.status);
            pi = k.pos4[i];
            beg = k.nbr_off[i]; end = use_far ? k.nbr_off[i + 1] : beg + k.nbr_near[i];
        }
        // compact lists: lane q < 27 holds the first atom of the q-th cell around the atom's build-time cell
        const int cs = (k.nbr16 && have && lane < 27) ? k.cell_start[neighbor_cell(k.grid, k.cell_id[i], lane)] : 0;
        auto entry = [&](int64_t e, bool live) {   // index of list entry e (every lane of the warp calls this together)
            if (!k.nbr16) return live ? (int)MLIP_CHECK_INDEX(k.nbr[MLIP_CHECK_INDEX(e, k.nbr_cap, k.status)], k.n, k.status) : 0;
            const int code = live ? k.nbr16[MLIP_CHECK_INDEX(e, k.nbr_cap, k.status)] : 0;
            const int base = __shfl_sync(0xffffffffu, cs, code >> L16_SHIFT);
            return live ? (int)MLIP_CHECK_INDEX(base + (code & L16_MASK), k.n, k.status) : 0;
        };

        // ---------------- Encoding: P = H^T G (Eq. 4) ----------------
        // Four pairs per m8n8k4 step on the fp64 tensor pipe.  A = H^T (rows = angular components, k = pair), B = G
        // (k = pair, columns = channels): lane (g, t) evaluates g of pair t at channels 16 q + 2 g, + 1 (q < K / 16), so the
        // eight lanes of a pair read 128 contiguous bytes of a table row per load and four rows are in flight per step; the
        // accumulators go through shared memory to lane = channel afterwards.
        constexpr int MT = (D + 7) / 8, NTK = K / 8, PS = 36;   // PS = 4 mod 16 doubles: the A-fragment reads fall on 32 different banks
        double P[D][CPL];
#pragma unroll
        for (int a = 0; a < D; ++a)
#pragma unroll
            for (int q = 0; q < CPL; ++q) P[a][q] = 0.0;
        int n_mine = 0;   // pairs of this warp's atom inside r_cut
        {
            double Pc[MT][NTK][2];
    #pragma unroll
            for (int mt = 0; mt < MT; ++mt)
    #pragma unroll
                for (int nt = 0; nt < NTK; ++nt) Pc[mt][nt][0] = Pc[mt][nt][1] = 0.0;
            double *hs = sm.pw[wid].te, *bq = hs + D * PS, *offs = bq + 4 * PS;
            for (int64_t base = beg; base < end; base += 32) {
                const int64_t e = base + lane;
                const int j_e = entry(e, e < end);
                bool valid = false;
                double dx = 0.0, dy = 0.0, dz = 0.0, d2 = 1.0;
                int sj = 0;
                if (e < end) {
                    const double4 pj = k.pos4[j_e];
                    dx = min_image(pj.x - pi.x, k.grid.box[0], k.grid.half[0]);
                    dy = min_image(pj.y - pi.y, k.grid.box[1], k.grid.half[1]);
                    dz = min_image(pj.z - pi.z, k.grid.box[2], k.grid.half[2]);
                    d2 = dx * dx + dy * dy + dz * dz;
                    sj = (int)pj.w;
                    valid = d2 < k.rc2;
                }
                const unsigned mask = __ballot_sync(0xffffffffu, valid);
                const int nv = __popc(mask);
                if (valid) {   // the pairs inside r_cut take consecutive columns of the hand-over rows
                    const int col = __popc(mask & ((1u << lane) - 1u));
                    if (n_mine + col < F64_QCAP) sm.q[wid][n_mine + col] = j_e;
                    const double r = sqrt(d2), rinv = 1.0 / r;
                    double h[D > D_ANG ? D : D_ANG], b[4];
                    if (CLOSED) harmonics(dx * rinv, dy * rinv, dz * rinv, h);
                    else angular_values<LMAX, BASIS>(dx * rinv, dy * rinv, dz * rinv, h);
                    const int iv = spline_basis<false, double>(r, k.r_min, k.inv_h, k.knots, b, nullptr, k.status);
    #pragma unroll
                    for (int a = 0; a < D; ++a) hs[a * PS + col] = h[a];
    #pragma unroll
                    for (int m = 0; m < 4; ++m) bq[m * PS + col] = b[m];
                    offs[col] = __longlong_as_double(((long long)(si * C + sj) * (k.knots + 3) + iv) * K);
                }
                n_mine += nv;
                __syncwarp();
                pc.mark(0);
                for (int p0 = 0; p0 < nv; p0 += 4) {
                    const int p = p0 + t;
                    const bool live = p < nv;   // a step past the last pair contracts zeros against the table's first rows
                    const double *cf = k.coef + (live ? __double_as_longlong(offs[p]) : 0ll) + 2 * g;
                    double gq[NTK];
#pragma unroll
                    for (int nt = 0; nt < NTK; ++nt) gq[nt] = 0.0;
#pragma unroll
                    for (int m = 0; m < 4; ++m) {
                        const double bm = live ? bq[m * PS + p] : 0.0;
                        double cc[NTK];
#pragma unroll
                        for (int v = 0; v < NTK; v += 2)   // 16 bytes per lane: the eight lanes of a pair read 128 contiguous bytes
                            asm volatile("ld.global.nc.v2.f64 {%0,%1}, [%2];" : "=d"(cc[v]), "=d"(cc[v + 1]) : "l"(cf + m * K + 8 * v));
#pragma unroll
                        for (int nt = 0; nt < NTK; ++nt) gq[nt] = fma(bm, cc[nt], gq[nt]);
                    }
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) {
                        const double av = (live && 8 * mt + g < D) ? hs[(8 * mt + g) * PS + p] : 0.0;
    #pragma unroll
                        for (int nt = 0; nt < NTK; ++nt) dmma(Pc[mt][nt][0], Pc[mt][nt][1], av, gq[nt]);
                    }
                }
                __syncwarp();
                pc.mark(1);
            }
            // fragments -> lane = channel: column n of n-tile nt is channel 16 (nt / 2) + 2 n + nt % 2
            double *pm = sm.pw[wid].w;
    #pragma unroll
            for (int mt = 0; mt < MT; ++mt)
    #pragma unroll
                for (int nt = 0; nt < NTK; ++nt)
    #pragma unroll
                    for (int u = 0; u < 2; ++u)
                        if (8 * mt + g < D) pm[(8 * mt + g) * K + 16 * (nt >> 1) + 2 * (2 * t + u) + (nt & 1)] = Pc[mt][nt][u];
            __syncwarp();
    #pragma unroll
            for (int q = 0; q < CPL; ++q) {
                const int c = lane + 32 * q;
                if (c < K) {
    #pragma unroll
                    for (int a = 0; a < D; ++a) P[a][q] = pm[a * K + c];
                }
            }
            __syncwarp();   // W_i is written over the same buffer below
        }

        n_pairs += n_mine;
        // ---------------- Invariants (Eq. 5: p^T C_l p); an empty slot of a ragged tile feeds zeros ----------------
#pragma unroll
        for (int q = 0; q < CPL; ++q) {
            const int c = lane + 32 * q;
            if (c < K) {
                sm.x[wid][c] = P[0][q];
#pragma unroll
                for (int l = 1; l <= LMAX; ++l) {
                    double s = 0.0;
#pragma unroll
                    for (int a = Shape::begin(l); a < Shape::begin(l + 1); ++a) s = fma(Shape::metric(a) * P[a][q], P[a][q], s);
                    sm.x[wid][l * K + c] = s;
                }
            }
        }
        pc.mark(2);
        __syncthreads();
        pc.mark(3);

        // ---------------- Regression (Eq. 6) and its reverse pass: the CTA on the tile ----------------
        {
            const int n = 8 * wid + g;   // this lane's row of W (forward: neuron; reverse: input of the layer)
            double y0, y1, d0, d1;
            {   // layer 0: pre[64 x 8] = W0 [64 x NINV] X^T
                double c0 = hd[H.bias + n], c1 = c0;
                const double *wrow = hd + H.w0 + (size_t)n * NINV + 4 * t;
                const double *xb = &sm.x[g][4 * t];
                constexpr int HS = (NINV / 16) % 2 == 0 ? 2 : 1;   // 16-input blocks per call
#pragma unroll 1
                for (int h0 = 0; h0 < NINV / 16; h0 += HS) head_dot<HS>(c0, c1, wrow + 16 * h0, xb + 16 * h0);
                y0 = silu_d(c0, d0); y1 = silu_d(c1, d1);
                sm.y[0][2 * t][n] = y0; sm.y[0][2 * t + 1][n] = y1;
                sm.sd[0][2 * t][n] = d0; sm.sd[0][2 * t + 1][n] = d1;
            }
            __syncthreads();
#pragma unroll 1
            for (int L = 1; L < HEAD_L; ++L) {
                double c0 = hd[H.bias + L * HEAD_H + n], c1 = c0;
                head_dot<HEAD_H / 16>(c0, c1, hd + H.wl + (L - 1) * HEAD_H * HEAD_H + n * HEAD_H + 4 * t, &sm.y[(L - 1) & 1][g][4 * t]);
                y0 += silu_d(c0, d0); y1 += silu_d(c1, d1);
                sm.y[L & 1][2 * t][n] = y0; sm.y[L & 1][2 * t + 1][n] = y1;
                sm.sd[L][2 * t][n] = d0; sm.sd[L][2 * t + 1][n] = d1;
                __syncthreads();
            }
            {   // output layer: warp = atom
                const double *yf = sm.y[(HEAD_L - 1) & 1][wid];
                double e_i = hd[H.wout + lane] * yf[lane] + hd[H.wout + 32 + lane] * yf[lane + 32];
#pragma unroll
                for (int o = 16; o; o >>= 1) e_i += __shfl_xor_sync(0xffffffffu, e_i, o);
                e_i += hd[H.wout + HEAD_H];
                if (lane == 0 && have) { k.e_atom[i] = e_i; e_sum += e_i; }
            }
            // reverse: this lane keeps dE/dy[n] of atoms 2t, 2t + 1; each hidden layer adds W^T (dE/dy . SiLU') through its
            // skip.  The transposed copies make the reverse pass read weight rows exactly as the forward pass does.
            double g0 = hd[H.wout + n], g1 = g0;
            sm.dp[(HEAD_L - 1) & 1][2 * t][n] = g0 * sm.sd[HEAD_L - 1][2 * t][n];
            sm.dp[(HEAD_L - 1) & 1][2 * t + 1][n] = g1 * sm.sd[HEAD_L - 1][2 * t + 1][n];
            __syncthreads();
#pragma unroll 1
            for (int L = HEAD_L - 1; L >= 1; --L) {
                head_dot<HEAD_H / 16>(g0, g1, hd + H.wlt + (L - 1) * HEAD_H * HEAD_H + n * HEAD_H + 4 * t, &sm.dp[L & 1][g][4 * t]);
                sm.dp[(L - 1) & 1][2 * t][n] = g0 * sm.sd[L - 1][2 * t][n];
                sm.dp[(L - 1) & 1][2 * t + 1][n] = g1 * sm.sd[L - 1][2 * t + 1][n];
                __syncthreads();
            }
            // layer 0: dE/dG [NINV x 8] = W0^T dp, written over the invariants; warp = every 8th block of 8 inputs
#pragma unroll 1
            for (int m = wid; m < NINV / 8; m += F64_TILE) {
                double c0 = 0.0, c1 = 0.0;
                head_dot<HEAD_H / 16>(c0, c1, hd + H.w0t + (size_t)(8 * m + g) * HEAD_H + 4 * t, &sm.dp[0][g][4 * t]);
                sm.x[2 * t][8 * m + g] = c0; sm.x[2 * t + 1][8 * m + g] = c1;
            }
            __syncthreads();
        }

        pc.mark(4);
        // W_i = dE_i/dP_i (Eq. 7)
        double *wi = sm.pw[wid].w;
#pragma unroll
        for (int q = 0; q < CPL; ++q) {
            const int c = lane + 32 * q;
            if (c < K) {
                wi[c] = sm.x[wid][c];
#pragma unroll
                for (int a = 1; a < D; ++a) wi[a * K + c] = (2.0 * Shape::metric(a)) * sm.x[wid][Shape::l_of(a) * K + c] * P[a][q];
            }
        }
        __syncwarp();

        // ---------------- Derivation (Eq. 8-10) ----------------
        // The pairs inside r_cut wait in the queue the encoding filled (a longer list is scanned again into a ring) and are
        // taken NB at a time.
        //   [V; T] = [G; G'] W^T (Eq. 9 and the re-associated Eq. 8 term) on the fp64 tensor pipe, 8 pairs per m8n8k4 tile:
        //   lane (g, t) evaluates g, g' of pair g at channels 16 h + 4 t .. + 3 straight into the A operand (the quad reads
        //   128 contiguous bytes of each table row), W_i sits in registers as B fragments, the accumulators return through
        //   shared memory to lane = pair for the projection.  16 pairs per batch: the staging rows share the hand-over
        //   buffer with W_i's shared-memory copy, which is dead once the fragments are loaded.
        constexpr int NB = 16;
        constexpr int NT = (D + 7) / 8;            // n-tiles of the tensor form
        constexpr int BS = 10, VTS = 2 * 8 * NT + 2;   // staging rows: 4 b, 4 b', table offset | V then T (+ 2: lane = pair reads 16
                                                       // bytes at a 68-word stride, eight lanes on 32 different banks)
        static_assert(NB * (BS + VTS) * sizeof(double) <= sizeof(sm.pw[0]), "derivation staging must fit the hand-over buffer");
        double fx = 0.0, fy = 0.0, fz = 0.0;
        int nq = 0, qh = 0;                        // ring: nq indices from position qh
        int *queue = sm.q[wid];
        double Bf[NT][K / 4];
        {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int ks = 0; ks < K / 4; ++ks)   // k-step ks = 4 h + u contracts channel 16 h + 4 t + u (see the loads below)
                    Bf[nt][ks] = (8 * nt + g < D) ? wi[(8 * nt + g) * K + 16 * (ks >> 2) + 4 * t + (ks & 3)] : 0.0;
            __syncwarp();   // from here on the buffer that held W_i is staging space
        }
        double *bs = reinterpret_cast<double *>(&sm.pw[wid]), *vt = bs + NB * BS;

        pc.mark(5);
        auto process = [&](int nb) {
            pc.mark(6);
            const int j = lane < nb ? queue[(qh + lane) & (F64_QCAP - 1)] : 0;
            double x = 0.0, y = 0.0, z = 0.0, rinv = 0.0, ux = 0.0, uy = 0.0, uz = 0.0;
            double b[4] = {0.0, 0.0, 0.0, 0.0}, db[4] = {0.0, 0.0, 0.0, 0.0};
            const double *cf = k.coef;
            if (lane < nb) {
                const double4 pj = k.pos4[j];
                x = min_image(pj.x - pi.x, k.grid.box[0], k.grid.half[0]);
                y = min_image(pj.y - pi.y, k.grid.box[1], k.grid.half[1]);
                z = min_image(pj.z - pi.z, k.grid.box[2], k.grid.half[2]);
                const double r = sqrt(x * x + y * y + z * z);
                rinv = 1.0 / r;
                ux = x * rinv; uy = y * rinv; uz = z * rinv;
                const int iv = spline_basis<true, double>(r, k.r_min, k.inv_h, k.knots, b, db, k.status);
                cf = k.coef + ((size_t)(si * C + (int)pj.w) * (k.knots + 3) + iv) * K;
            }
            double s = 0.0, tx = 0.0, ty = 0.0, tz = 0.0, tu = 0.0;
            {
                if (lane < NB) {   // hand the spline weights and the table row to the tile's lanes
                    double *row = bs + lane * BS;
#pragma unroll
                    for (int m = 0; m < 4; ++m) { row[m] = b[m]; row[4 + m] = db[m]; }
                    row[8] = __longlong_as_double((long long)(cf - k.coef));
                }
                __syncwarp();
                pc.mark(7);
#pragma unroll 1
                for (int grp = 0; grp < NB / 8; ++grp) {
                    if (8 * grp >= nb) break;
                    const double *row = bs + (8 * grp + g) * BS;
                    double wb[4], wd[4];
#pragma unroll
                    for (int m = 0; m < 4; ++m) { wb[m] = row[m]; wd[m] = row[4 + m]; }
                    const double *ct = k.coef + __double_as_longlong(row[8]) + 4 * t;
                    double V[NT][2], T[NT][2];
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) { V[nt][0] = V[nt][1] = T[nt][0] = T[nt][1] = 0.0; }
                    // the channel <-> k-index assignment is free (both operands use it); with lane t on channels
                    // 16 h + 4 t .. + 3 the quad reads 128 contiguous bytes of a table row per load
#pragma unroll
                    for (int h = 0; h < K / 16; ++h) {
                        double gv[4] = {0.0, 0.0, 0.0, 0.0}, dg[4] = {0.0, 0.0, 0.0, 0.0};
#pragma unroll
                        for (int m = 0; m < 4; ++m) {
                            double cc[4];
                            asm volatile("ld.global.nc.v4.f64 {%0,%1,%2,%3}, [%4];"
                                         : "=d"(cc[0]), "=d"(cc[1]), "=d"(cc[2]), "=d"(cc[3]) : "l"(ct + m * K + 16 * h));
#pragma unroll
                            for (int u = 0; u < 4; ++u) { gv[u] = fma(wb[m], cc[u], gv[u]); dg[u] = fma(wd[m], cc[u], dg[u]); }
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u)
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt) {
                                dmma(V[nt][0], V[nt][1], gv[u], Bf[nt][4 * h + u]);
                                dmma(T[nt][0], T[nt][1], dg[u], Bf[nt][4 * h + u]);
                            }
                    }
                    double *out = vt + (8 * grp + g) * VTS + 2 * t;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        *reinterpret_cast<double2 *>(out + 8 * nt) = make_double2(V[nt][0], V[nt][1]);
                        *reinterpret_cast<double2 *>(out + 8 * NT + 8 * nt) = make_double2(T[nt][0], T[nt][1]);
                    }
                }
                __syncwarp();
                pc.mark(8);
                if (lane < nb) {
                    if constexpr (CLOSED) {
                        double v[D_ANG], tt[D_ANG];   // components beyond d are zero and drop out of the projection
                        const double *rowv = vt + lane * VTS;
#pragma unroll
                        for (int a = 0; a < D_ANG; a += 2) {
                            double2 pv = make_double2(0.0, 0.0), pt = pv;
                            if (a < 8 * NT) { pv = *reinterpret_cast<const double2 *>(rowv + a); pt = *reinterpret_cast<const double2 *>(rowv + 8 * NT + a); }
                            v[a] = pv.x; v[a + 1] = pv.y; tt[a] = pt.x; tt[a + 1] = pt.y;
                        }
                        harmonics_project(ux, uy, uz, v, tt, s, tx, ty, tz, tu);
                    } else {
                        // the rows of the angular degrees L0 .. L1 projected at once; wide bases go through in two degree
                        // ranges so that v and t stay in registers
                        const double *rowv = vt + lane * VTS;
                        auto rows_of = [&](auto l0c, auto l1c) {
                            constexpr int L0 = decltype(l0c)::value, L1 = decltype(l1c)::value;
                            constexpr int A0 = Shape::begin(L0), A1 = Shape::begin(L1 + 1);
                            constexpr int DV = A1 - A0;
                            double v[DV], tt[DV];
#pragma unroll
                            for (int a = 0; a < DV; ++a) { v[a] = rowv[A0 + a]; tt[a] = rowv[8 * NT + A0 + a]; }
                            double ps, px, py, pz, pu;
                            angular_project<LMAX, BASIS, L0, L1>(ux, uy, uz, v, tt, ps, px, py, pz, pu);
                            s += ps; tx += px; ty += py; tz += pz; tu += pu;
                        };
                        if constexpr (D > 25) {
                            rows_of(std::integral_constant<int, 0>{}, std::integral_constant<int, 3>{});
                            rows_of(std::integral_constant<int, 4>{}, std::integral_constant<int, LMAX>{});
                        } else {
                            rows_of(std::integral_constant<int, 0>{}, std::integral_constant<int, LMAX>{});
                        }
                    }
                }
                __syncwarp();
            }
            if (lane < nb) {
                // f_ij = (g' . u_ij) r^ + J_ang^T v_ij,  J_ang = (grad_u h)(I - u u^T) / r
                const double qx = s * ux + (tx - tu * ux) * rinv;
                const double qy = s * uy + (ty - tu * uy) * rinv;
                const double qz = s * uz + (tz - tu * uz) * rinv;
                fx += qx; fy += qy; fz += qz;
                atomicAdd(&k.force[3 * (size_t)j], -qx);
                atomicAdd(&k.force[3 * (size_t)j + 1], -qy);
                atomicAdd(&k.force[3 * (size_t)j + 2], -qz);
                vir[0] -= x * qx; vir[1] -= x * qy; vir[2] -= x * qz;
                vir[3] -= y * qx; vir[4] -= y * qy; vir[5] -= y * qz;
                vir[6] -= z * qx; vir[7] -= z * qy; vir[8] -= z * qz;
            }
            qh = (qh + nb) & (F64_QCAP - 1);
            nq -= nb;
            pc.mark(9);
        };

        // one loop for both cases: with every pair already queued there is nothing to scan
        const bool kept = n_mine <= F64_QCAP;
        if (kept) nq = n_mine;
        for (int64_t base = kept ? end : beg;;) {
            if (base < end) {   // compact the next 32 list entries' pairs inside r_cut into the ring
                const int64_t e = base + lane;
                bool valid = false;
                const int j = entry(e, e < end);
                if (e < end) {
                    const double4 pj = k.pos4[j];
                    const double dx = min_image(pj.x - pi.x, k.grid.box[0], k.grid.half[0]);
                    const double dy = min_image(pj.y - pi.y, k.grid.box[1], k.grid.half[1]);
                    const double dz = min_image(pj.z - pi.z, k.grid.box[2], k.grid.half[2]);
                    valid = dx * dx + dy * dy + dz * dz < k.rc2;
                }
                const unsigned m = __ballot_sync(0xffffffffu, valid);
                if (valid) queue[(qh + nq + __popc(m & ((1u << lane) - 1u))) & (F64_QCAP - 1)] = j;
                nq += __popc(m);
                base += 32;
                __syncwarp();
            }
            const bool last = base >= end;
            while (nq >= NB || (last && nq > 0)) { process(min(nq, NB)); __syncwarp(); }
            if (last) break;
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            fx += __shfl_xor_sync(0xffffffffu, fx, o);
            fy += __shfl_xor_sync(0xffffffffu, fy, o);
            fz += __shfl_xor_sync(0xffffffffu, fz, o);
        }
        if (lane == 0 && have) {
            atomicAdd(&k.force[3 * (size_t)i], fx);
            atomicAdd(&k.force[3 * (size_t)i + 1], fy);
            atomicAdd(&k.force[3 * (size_t)i + 2], fz);
        }
        pc.mark(6);
        __syncthreads();   // the next tile's encoding reuses the hand-over rows that alias W_i, and x
        pc.mark(10);
    }
    pc.flush(k.acc, lane);

#pragma unroll
    for (int q = 0; q < 9; ++q) {
        double x = vir[q];
#pragma unroll
        for (int o = 16; o; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
        if (lane == 0) atomicAdd(&k.acc[ACC_VIRIAL + q], x);
    }
    if (lane == 0) {
        atomicAdd(&k.acc[ACC_ENERGY], e_sum);
        atomicAdd(k.pair_counter, n_pairs);
    }
}

// fp64 forces and energies -> the fp32 arrays the fp32 getters read
__global__ void k_force_to_float(int64_t n, const double *__restrict__ fd, const double *__restrict__ ed, float4 *__restrict__ force,
                                 float *__restrict__ e_atom) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    force[i] = make_float4((float)fd[3 * i], (float)fd[3 * i + 1], (float)fd[3 * i + 2], 0.f);
    e_atom[i] = (float)ed[i];
}

int upload_head_f64(mlip_ctx *c, const double *w) {
    const int C = c->cfg.n_species, n_inv = (c->cfg.l_max + 1) * c->cfg.k;
    const Head64 H(n_inv);
    const size_t net = head_net_size(n_inv);
    double *host = (double *)calloc((size_t)C * H.total, sizeof(double));
    if (!host) return MLIP_ERR_OOM;
    for (int s = 0; s < C; ++s) {
        const double *src = w + (size_t)s * net;
        double *hp = host + (size_t)s * H.total;
        int in = n_inv;
        for (int L = 0; L < HEAD_L; ++L) {
            double *row = L == 0 ? hp + H.w0 : hp + H.wl + (L - 1) * HEAD_H * HEAD_H;
            memcpy(row, src, sizeof(double) * HEAD_H * in);
            double *tr = L == 0 ? hp + H.w0t : hp + H.wlt + (L - 1) * HEAD_H * HEAD_H;   // [in][64]
            for (int o = 0; o < HEAD_H; ++o)
                for (int q = 0; q < in; ++q) tr[(size_t)q * HEAD_H + o] = src[(size_t)o * in + q];
            memcpy(hp + H.bias + L * HEAD_H, src + in * HEAD_H, sizeof(double) * HEAD_H);
            src += in * HEAD_H + HEAD_H;
            in = HEAD_H;
        }
        memcpy(hp + H.wout, src, sizeof(double) * (HEAD_H + 1));
    }
    const size_t bytes = sizeof(double) * (size_t)C * H.total;
    cudaError_t e = cudaMalloc(&c->head_w_d, bytes);
    if (e == cudaSuccess) e = cudaMemcpy(c->head_w_d, host, bytes, cudaMemcpyHostToDevice);
    free(host);
    if (e != cudaSuccess) { c->err = cudaGetErrorString(e); return MLIP_ERR_CUDA; }
    c->resident += bytes;
    return MLIP_OK;
}

template <int K, int LMAX, int BASIS>
static cudaError_t launch_shape(mlip_ctx *c, const F64Args &k, cudaStream_t s, cudaEvent_t start, cudaEvent_t stop) {
    const size_t smem_bytes = sizeof(TileSmem<K, LMAX, BASIS>);
    if (!c->kernel_ready) {
        cudaError_t e = cudaFuncSetAttribute(k_mega_f64<K, LMAX, BASIS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
        if (e != cudaSuccess) return e;
        if (!(BASIS == 0 && LMAX <= 3)) {   // projection matrices for the general angular routines
            double q[Q_TOTAL];
            build_q_tables(q);
            e = cudaMemcpyToSymbol(c_ang_q, q, sizeof q);
            if (e != cudaSuccess) return e;
        }
        c->kernel_ready = true;
    }
    const int per_sm = f64_ctas_per_sm<K, LMAX, BASIS>();
    const int64_t tiles_max = (k.n + F64_TILE - 1) / F64_TILE + k.n_species;
    const int blocks = (int)std::min<int64_t>(tiles_max, (int64_t)per_sm * c->n_sm);
    cudaEventRecord(start, s);
    k_mega_f64<K, LMAX, BASIS><<<blocks, F64_TILE * 32, smem_bytes, s>>>(k);
    cudaEventRecord(stop, s);
    return cudaGetLastError();
}

bool f64_shape_supported(int k, int l_max, int basis) {
    if (basis == 0 && (k == 16 || k == 32 || k == 64) && l_max >= 1 && l_max <= 3) return true;
    if (basis == 0 && k == 32 && (l_max == 4 || l_max == 5)) return true;
    if (basis == 1 && (k == 32 || k == 64) && l_max >= 1 && l_max <= 3) return true;
    return false;
}

int launch_megakernel_f64(mlip_ctx *c, cudaStream_t s) {
    const int64_t n = c->n;
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->force_d, 0, sizeof(double) * 3 * n, s));
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->launch_block, 0, LAUNCH_CLEAR_BYTES, s));   // pair counter and accumulators
    F64Args k;
    k.n = n; k.n_species = c->cfg.n_species; k.grid = c->grid; k.rc2 = c->cfg.r_cut * c->cfg.r_cut;
    k.coef = c->table_d; k.knots = c->cfg.table_knots; k.r_min = c->cfg.table_r_min;
    k.inv_h = c->cfg.table_knots / (c->cfg.r_cut - c->cfg.table_r_min);
    k.pos4 = c->pos4; k.center_order = c->center_order; k.species_start = c->species_start;
    k.nbr_off = c->nbr_off; k.nbr_near = c->nbr_near; k.far_flag = c->far_flag; k.nbr = c->nbr; k.nbr16 = c->list16 ? reinterpret_cast<const uint16_t *>(c->nbr) : nullptr; k.cell_id = c->cell_id; k.cell_start = c->cell_start;
    k.nbr_cap = c->nbr_cap;
    k.head = c->head_w_d; k.force = c->force_d; k.e_atom = c->e_atom_d; k.acc = c->acc;
    k.pair_counter = c->pair_counter; k.status = c->status;
    const int slot = (int)(c->ev_count % mlip_ctx::EV_POOL);
    cudaEvent_t e0 = c->ev[2 * slot], e1 = c->ev[2 * slot + 1];
    cudaError_t e = cudaErrorInvalidValue;
    switch (c->cfg.basis * 1000 + c->cfg.k * 10 + c->cfg.l_max) {
#define MLIP_F64_CASE(K, L, B) case B * 1000 + K * 10 + L: e = launch_shape<K, L, B>(c, k, s, e0, e1); break;
        MLIP_F64_CASE(16, 1, 0) MLIP_F64_CASE(16, 2, 0) MLIP_F64_CASE(16, 3, 0)
        MLIP_F64_CASE(32, 1, 0) MLIP_F64_CASE(32, 2, 0) MLIP_F64_CASE(32, 3, 0)
        MLIP_F64_CASE(64, 1, 0) MLIP_F64_CASE(64, 2, 0) MLIP_F64_CASE(64, 3, 0)
        MLIP_F64_CASE(32, 4, 0) MLIP_F64_CASE(32, 5, 0)
        MLIP_F64_CASE(32, 1, 1) MLIP_F64_CASE(32, 2, 1) MLIP_F64_CASE(32, 3, 1)
        MLIP_F64_CASE(64, 1, 1) MLIP_F64_CASE(64, 2, 1) MLIP_F64_CASE(64, 3, 1)
#undef MLIP_F64_CASE
    }
    MLIP_CUDA_TRY(c, e);
    c->ev_count += 1;
    k_force_to_float<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(n, c->force_d, c->e_atom_d, c->force, c->e_atom);
    c->launches += 2;
    MLIP_CUDA_TRY(c, cudaGetLastError());
    return MLIP_OK;
}

}  // namespace mlip
