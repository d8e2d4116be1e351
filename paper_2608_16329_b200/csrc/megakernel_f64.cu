// Double-precision evaluation path (`precision = 1`): the same fused pass as megakernel.cu --
// encoding (Eq. 1-5), regression (Eq. 6) and derivation (Eq. 7-10) of an atom back to back with
// nothing per pair or per atom written to device memory except forces and E_i -- in plain fp64
// arithmetic.  Section 4.2 evaluates the potential in double precision by default; this path is
// for validation and for runs that want that accuracy.  The tensor pipe has no fp64 mode worth
// the operand shuffling at these shapes, so every contraction here is DFMA work:
//
//   one warp = one atom at a time (atoms in (species, cell) order, static stride over warps)
//   encoding    lane = list entry for geometry, harmonics and spline basis; then lane = channel
//               for g (Eq. 2) and the moment P (Eq. 4), the pair's h / basis handed over in
//               shared memory
//   regression  lane = neuron (and neuron + 32); weights read from L2 (a transposed copy for the
//               forward pass keeps both directions coalesced)
//   derivation  lane = pair, after compacting the pairs inside r_cut: v = W g, t = W g' against
//               W_i in shared memory, projection onto the pair vector, fp64 atomics for f_j
//
// The radial tables are the same clamped cubic B-splines as in the fp32 path but with fp64
// coefficients and enough knots for ~1e-11 relative error; they stay in global memory (L2).
//
// The kernel is a template over the descriptor shape: k in {16, 32, 64} radial channels and
// l_max in {1, 2, 3} (d = 4, 9, 16), the throughput side of the paper's ablations (Tables 6, 7 and
// Fig. 4(c)).  With k = 16 the upper half-warp idles in the lane = channel phases; with k = 64
// a lane owns channels lane and lane + 32.
#include <algorithm>

#include "common.cuh"
#include "pair_math.cuh"

namespace mlip {

constexpr int F64_WARPS = 8;
constexpr int F64_ST = 22;          // hand-over row: 16 h, 4 b, table offset, pad

// per-species head block (doubles) for n_inv inputs
struct Head64 {
    int w0, w0t, wl, wlt, bias, wout, total;
    __host__ __device__ constexpr explicit Head64(int n_inv)
        : w0(0),                                            // [64][n_inv]  row-major, reverse pass
          w0t(HEAD_H * n_inv),                              // [n_inv][64]  transposed, forward pass
          wl(2 * HEAD_H * n_inv),                           // 3 x [64][64]
          wlt(wl + (HEAD_L - 1) * HEAD_H * HEAD_H),
          bias(wlt + (HEAD_L - 1) * HEAD_H * HEAD_H),       // [4][64]
          wout(bias + HEAD_L * HEAD_H),                     // [64] + b_out
          total(wout + HEAD_H + 8) {}
};

__host__ __device__ constexpr int l_of(int a) { return a == 0 ? 0 : (a < 4 ? 1 : (a < 9 ? 2 : 3)); }

template <int K, int LMAX>
struct WarpScratch {
    static constexpr int D = (LMAX + 1) * (LMAX + 1);
    static constexpr int NINV = (LMAX + 1) * K;
    static constexpr int NINV_PAD = (NINV + 31) / 32 * 32;
    double x[NINV_PAD];           // invariants, then dE/dG
    double y[HEAD_H];             // running activation
    double sd[HEAD_L][HEAD_H];    // SiLU'(pre-activation) per layer
    double dp[HEAD_H];            // dE/dpre of the current layer
    double w[D * K];              // W_i = dE_i/dP_i (Eq. 7)
    double st[32][F64_ST];
    int q[64];                    // compacted neighbor indices
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
    const int64_t *nbr_off;
    const int32_t *nbr;
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

// One hidden layer forward for this warp's atom: pre = W in + b for neurons lane, lane + 32.
template <int IN>
__device__ __forceinline__ void layer_forward(const double *__restrict__ wt, const double *__restrict__ bias, const double *in, int lane,
                                              double &p0, double &p1) {
    p0 = bias[lane]; p1 = bias[lane + 32];
#pragma unroll 8
    for (int i = 0; i < IN; ++i) {
        const double a = in[i];
        p0 = fma(wt[i * HEAD_H + lane], a, p0);
        p1 = fma(wt[i * HEAD_H + 32 + lane], a, p1);
    }
}

template <int K, int LMAX>
__global__ void __launch_bounds__(F64_WARPS * 32, K <= 32 ? 2 : 1) k_mega_f64(F64Args k) {
    using WS = WarpScratch<K, LMAX>;
    constexpr int D = WS::D, NINV = WS::NINV, NQ = WS::NINV_PAD / 32;
    constexpr int CPL = (K + 31) / 32;   // channels per lane
    constexpr Head64 H(NINV);
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    WS &ws = reinterpret_cast<WS *>(smem_raw)[wid];
    const int C = k.n_species;
    const int64_t n_warps = (int64_t)gridDim.x * F64_WARPS;
    double e_sum = 0.0, vir[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};
    unsigned long long n_pairs = 0;

    for (int64_t slot = (int64_t)blockIdx.x * F64_WARPS + wid; slot < k.n; slot += n_warps) {
        const int i = k.center_order[slot];
        const double4 pi = k.pos4[i];
        const int si = (int)pi.w;
        const int64_t beg = k.nbr_off[i], end = k.nbr_off[i + 1];
        const double *hd = k.head + (size_t)si * H.total;

        // ---------------- Encoding: P = H^T G (Eq. 4), lane = channel ----------------
        double P[D][CPL];
#pragma unroll
        for (int a = 0; a < D; ++a)
#pragma unroll
            for (int q = 0; q < CPL; ++q) P[a][q] = 0.0;
        for (int64_t base = beg; base < end; base += 32) {
            const int64_t e = base + lane;
            bool valid = false;
            if (e < end) {
                const int j = k.nbr[e];
                const double4 pj = k.pos4[j];
                const double dx = min_image(pj.x - pi.x, k.grid.box[0], k.grid.half[0]);
                const double dy = min_image(pj.y - pi.y, k.grid.box[1], k.grid.half[1]);
                const double dz = min_image(pj.z - pi.z, k.grid.box[2], k.grid.half[2]);
                const double d2 = dx * dx + dy * dy + dz * dz;
                valid = d2 < k.rc2;
                if (valid) {
                    const double r = sqrt(d2), rinv = 1.0 / r;
                    double h[D_ANG], b[4];
                    harmonics(dx * rinv, dy * rinv, dz * rinv, h);
                    const int iv = spline_basis<false, double>(r, k.r_min, k.inv_h, k.knots, b, nullptr, k.status);
#pragma unroll
                    for (int a = 0; a < D; ++a) ws.st[lane][a] = h[a];
#pragma unroll
                    for (int m = 0; m < 4; ++m) ws.st[lane][16 + m] = b[m];
                    const long long off = ((long long)(si * C + (int)pj.w) * (k.knots + 3) + iv) * K;
                    ws.st[lane][20] = __longlong_as_double(off);
                }
            }
            unsigned mask = __ballot_sync(0xffffffffu, valid);
            n_pairs += __popc(mask);
            __syncwarp();
            while (mask) {
                const int p = __ffs(mask) - 1;
                mask &= mask - 1;
                const double *row = ws.st[p];
                const double *cf = k.coef + __double_as_longlong(row[20]);
#pragma unroll
                for (int q = 0; q < CPL; ++q) {
                    const int c = lane + 32 * q;
                    double g = 0.0;
                    if (c < K) {
                        g = row[16] * cf[c];
                        g = fma(row[17], cf[K + c], g);
                        g = fma(row[18], cf[2 * K + c], g);
                        g = fma(row[19], cf[3 * K + c], g);
                    }
#pragma unroll
                    for (int a = 0; a < D; ++a) P[a][q] = fma(row[a], g, P[a][q]);
                }
            }
            __syncwarp();
        }

        // ---------------- Invariants (Eq. 5, C_l = I) ----------------
#pragma unroll
        for (int q = 0; q < CPL; ++q) {
            const int c = lane + 32 * q;
            if (c < K) {
                ws.x[c] = P[0][q];
#pragma unroll
                for (int l = 1; l <= LMAX; ++l) {
                    double s = 0.0;
#pragma unroll
                    for (int a = l * l; a < (l + 1) * (l + 1); ++a) s = fma(P[a][q], P[a][q], s);
                    ws.x[l * K + c] = s;
                }
            }
        }
        __syncwarp();

        // ---------------- Regression (Eq. 6) and its reverse pass ----------------
        {
            double p0, p1, d0, d1;
            layer_forward<NINV>(hd + H.w0t, hd + H.bias, ws.x, lane, p0, p1);
            double y0 = silu_d(p0, d0), y1 = silu_d(p1, d1);
            ws.sd[0][lane] = d0; ws.sd[0][lane + 32] = d1;
            ws.y[lane] = y0; ws.y[lane + 32] = y1;
            __syncwarp();
#pragma unroll 1
            for (int L = 1; L < HEAD_L; ++L) {
                layer_forward<HEAD_H>(hd + H.wlt + (L - 1) * HEAD_H * HEAD_H, hd + H.bias + L * HEAD_H, ws.y, lane, p0, p1);
                y0 += silu_d(p0, d0); y1 += silu_d(p1, d1);
                __syncwarp();
                ws.sd[L][lane] = d0; ws.sd[L][lane + 32] = d1;
                ws.y[lane] = y0; ws.y[lane + 32] = y1;
                __syncwarp();
            }
            const double wo0 = hd[H.wout + lane], wo1 = hd[H.wout + 32 + lane];
            double e_i = wo0 * y0 + wo1 * y1;
#pragma unroll
            for (int o = 16; o; o >>= 1) e_i += __shfl_xor_sync(0xffffffffu, e_i, o);
            e_i += hd[H.wout + HEAD_H];
            if (lane == 0) { k.e_atom[i] = e_i; e_sum += e_i; }

            // dE/dy of the last layer is w_out; each hidden layer adds W^T (dE/dy . SiLU') through its skip
            double g0 = wo0, g1 = wo1;
#pragma unroll 1
            for (int L = HEAD_L - 1; L >= 1; --L) {
                ws.dp[lane] = g0 * ws.sd[L][lane]; ws.dp[lane + 32] = g1 * ws.sd[L][lane + 32];
                __syncwarp();
                const double *w = hd + H.wl + (L - 1) * HEAD_H * HEAD_H;
#pragma unroll 8
                for (int o = 0; o < HEAD_H; ++o) {
                    const double d = ws.dp[o];
                    g0 = fma(w[o * HEAD_H + lane], d, g0);
                    g1 = fma(w[o * HEAD_H + 32 + lane], d, g1);
                }
                __syncwarp();
            }
            ws.dp[lane] = g0 * ws.sd[0][lane]; ws.dp[lane + 32] = g1 * ws.sd[0][lane + 32];
            __syncwarp();
            double dx[NQ];   // dE/dG of invariants lane + 32 q
#pragma unroll
            for (int q = 0; q < NQ; ++q) dx[q] = 0.0;
            const double *w0 = hd + H.w0;
#pragma unroll 4
            for (int o = 0; o < HEAD_H; ++o) {
                const double d = ws.dp[o];
#pragma unroll
                for (int q = 0; q < NQ; ++q)
                    if (lane + 32 * q < NINV) dx[q] = fma(w0[o * NINV + 32 * q + lane], d, dx[q]);
            }
#pragma unroll
            for (int q = 0; q < NQ; ++q) ws.x[lane + 32 * q] = dx[q];
            __syncwarp();
            // W_i = dE_i/dP_i (Eq. 7)
#pragma unroll
            for (int q = 0; q < CPL; ++q) {
                const int c = lane + 32 * q;
                if (c < K) {
                    ws.w[c] = ws.x[c];
#pragma unroll
                    for (int a = 1; a < D; ++a) ws.w[a * K + c] = 2.0 * ws.x[l_of(a) * K + c] * P[a][q];
                }
            }
            __syncwarp();
        }

        // ---------------- Derivation (Eq. 8-10), lane = pair ----------------
        double fx = 0.0, fy = 0.0, fz = 0.0;
        int nq = 0;
        for (int64_t base = beg; base < end || nq > 0; base += 32) {
            if (base < end) {   // compact the entries inside r_cut into the warp's queue
                const int64_t e = base + lane;
                bool valid = false;
                int j = 0;
                if (e < end) {
                    j = k.nbr[e];
                    const double4 pj = k.pos4[j];
                    const double dx = min_image(pj.x - pi.x, k.grid.box[0], k.grid.half[0]);
                    const double dy = min_image(pj.y - pi.y, k.grid.box[1], k.grid.half[1]);
                    const double dz = min_image(pj.z - pi.z, k.grid.box[2], k.grid.half[2]);
                    valid = dx * dx + dy * dy + dz * dz < k.rc2;
                }
                const unsigned m = __ballot_sync(0xffffffffu, valid);
                if (valid) ws.q[nq + __popc(m & ((1u << lane) - 1u))] = j;
                nq += __popc(m);
                __syncwarp();
                if (nq < 32 && base + 32 < end) continue;
            }
            const int nb = min(nq, 32);
            if (lane < nb) {
                const int j = ws.q[lane];
                const double4 pj = k.pos4[j];
                const double x = min_image(pj.x - pi.x, k.grid.box[0], k.grid.half[0]);
                const double y = min_image(pj.y - pi.y, k.grid.box[1], k.grid.half[1]);
                const double z = min_image(pj.z - pi.z, k.grid.box[2], k.grid.half[2]);
                const double r = sqrt(x * x + y * y + z * z), rinv = 1.0 / r;
                const double ux = x * rinv, uy = y * rinv, uz = z * rinv;
                double b[4], db[4];
                const int iv = spline_basis<true, double>(r, k.r_min, k.inv_h, k.knots, b, db, k.status);
                const double *cf = k.coef + ((size_t)(si * C + (int)pj.w) * (k.knots + 3) + iv) * K;
                double v[D_ANG], t[D_ANG];   // components beyond d stay zero and drop out of the projection
#pragma unroll
                for (int a = 0; a < D_ANG; ++a) { v[a] = 0.0; t[a] = 0.0; }
#pragma unroll 1
                for (int c = 0; c < K; c += 2) {
                    double g0 = 0.0, g1 = 0.0, dg0 = 0.0, dg1 = 0.0;
#pragma unroll
                    for (int m = 0; m < 4; ++m) {
                        const double2 cc = *reinterpret_cast<const double2 *>(cf + m * K + c);
                        g0 = fma(b[m], cc.x, g0); g1 = fma(b[m], cc.y, g1);
                        dg0 = fma(db[m], cc.x, dg0); dg1 = fma(db[m], cc.y, dg1);
                    }
#pragma unroll
                    for (int a = 0; a < D; ++a) {
                        const double2 w = *reinterpret_cast<const double2 *>(&ws.w[a * K + c]);
                        v[a] = fma(w.x, g0, fma(w.y, g1, v[a]));
                        t[a] = fma(w.x, dg0, fma(w.y, dg1, t[a]));
                    }
                }
                double s, tx, ty, tz, tu;
                harmonics_project(ux, uy, uz, v, t, s, tx, ty, tz, tu);
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
            __syncwarp();
            // move what is left of the queue to its front
            const int rest = nq - nb;
            const int keep = lane < rest ? ws.q[nb + lane] : 0;
            __syncwarp();
            if (lane < rest) ws.q[lane] = keep;
            nq = rest;
            __syncwarp();
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            fx += __shfl_xor_sync(0xffffffffu, fx, o);
            fy += __shfl_xor_sync(0xffffffffu, fy, o);
            fz += __shfl_xor_sync(0xffffffffu, fz, o);
        }
        if (lane == 0) {
            atomicAdd(&k.force[3 * (size_t)i], fx);
            atomicAdd(&k.force[3 * (size_t)i + 1], fy);
            atomicAdd(&k.force[3 * (size_t)i + 2], fz);
        }
    }

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
            double *tr = L == 0 ? hp + H.w0t : hp + H.wlt + (L - 1) * HEAD_H * HEAD_H;
            for (int o = 0; o < HEAD_H; ++o)
                for (int q = 0; q < in; ++q) {
                    row[o * in + q] = src[o * in + q];
                    tr[q * HEAD_H + o] = src[o * in + q];
                }
            for (int o = 0; o < HEAD_H; ++o) hp[H.bias + L * HEAD_H + o] = src[in * HEAD_H + o];
            src += in * HEAD_H + HEAD_H;
            in = HEAD_H;
        }
        for (int o = 0; o < HEAD_H + 1; ++o) hp[H.wout + o] = src[o];
    }
    const size_t bytes = sizeof(double) * (size_t)C * H.total;
    cudaError_t e = cudaMalloc(&c->head_w_d, bytes);
    if (e == cudaSuccess) e = cudaMemcpy(c->head_w_d, host, bytes, cudaMemcpyHostToDevice);
    free(host);
    if (e != cudaSuccess) { c->err = cudaGetErrorString(e); return MLIP_ERR_CUDA; }
    c->resident += bytes;
    return MLIP_OK;
}

template <int K, int LMAX>
static cudaError_t launch_shape(mlip_ctx *c, const F64Args &k, cudaStream_t s, cudaEvent_t start, cudaEvent_t stop) {
    const size_t smem_bytes = sizeof(WarpScratch<K, LMAX>) * F64_WARPS;
    if (!c->kernel_ready) {
        cudaError_t e = cudaFuncSetAttribute(k_mega_f64<K, LMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
        if (e != cudaSuccess) return e;
        c->kernel_ready = true;
    }
    const int per_sm = K <= 32 ? 2 : 1;
    const int blocks = (int)std::min<int64_t>((k.n + F64_WARPS - 1) / F64_WARPS, (int64_t)per_sm * c->n_sm);
    cudaEventRecord(start, s);
    k_mega_f64<K, LMAX><<<blocks, F64_WARPS * 32, smem_bytes, s>>>(k);
    cudaEventRecord(stop, s);
    return cudaGetLastError();
}

bool f64_shape_supported(int k, int l_max) { return (k == 16 || k == 32 || k == 64) && l_max >= 1 && l_max <= 3; }

int launch_megakernel_f64(mlip_ctx *c, cudaStream_t s) {
    const int64_t n = c->n;
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->force_d, 0, sizeof(double) * 3 * n, s));
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->acc, 0, sizeof(double) * ACC_KINETIC, s));
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->pair_counter, 0, sizeof(unsigned long long), s));
    F64Args k;
    k.n = n; k.n_species = c->cfg.n_species; k.grid = c->grid; k.rc2 = c->cfg.r_cut * c->cfg.r_cut;
    k.coef = c->table_d; k.knots = c->cfg.table_knots; k.r_min = c->cfg.table_r_min;
    k.inv_h = c->cfg.table_knots / (c->cfg.r_cut - c->cfg.table_r_min);
    k.pos4 = c->pos4; k.center_order = c->center_order; k.nbr_off = c->nbr_off; k.nbr = c->nbr;
    k.head = c->head_w_d; k.force = c->force_d; k.e_atom = c->e_atom_d; k.acc = c->acc;
    k.pair_counter = c->pair_counter; k.status = c->status;
    const int slot = (int)(c->ev_count % mlip_ctx::EV_POOL);
    cudaEvent_t e0 = c->ev[2 * slot], e1 = c->ev[2 * slot + 1];
    cudaError_t e = cudaErrorInvalidValue;
    switch (c->cfg.k * 10 + c->cfg.l_max) {
#define MLIP_F64_CASE(K, L) case K * 10 + L: e = launch_shape<K, L>(c, k, s, e0, e1); break;
        MLIP_F64_CASE(16, 1) MLIP_F64_CASE(16, 2) MLIP_F64_CASE(16, 3)
        MLIP_F64_CASE(32, 1) MLIP_F64_CASE(32, 2) MLIP_F64_CASE(32, 3)
        MLIP_F64_CASE(64, 1) MLIP_F64_CASE(64, 2) MLIP_F64_CASE(64, 3)
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
