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
#include <algorithm>

#include "common.cuh"
#include "pair_math.cuh"

namespace mlip {

constexpr int F64_WARPS = 8;
constexpr int F64_ST = 22;          // hand-over row: 16 h, 4 b, table offset, pad

// per-species head block (doubles)
constexpr int H64_W0 = 0;                                   // [64][128]  row-major, reverse pass
constexpr int H64_W0T = H64_W0 + HEAD_H * N_INV;            // [128][64]  transposed, forward pass
constexpr int H64_WL = H64_W0T + HEAD_H * N_INV;            // 3 x [64][64]
constexpr int H64_WLT = H64_WL + (HEAD_L - 1) * HEAD_H * HEAD_H;
constexpr int H64_BIAS = H64_WLT + (HEAD_L - 1) * HEAD_H * HEAD_H;   // [4][64]
constexpr int H64_WOUT = H64_BIAS + HEAD_L * HEAD_H;        // [64] + b_out
constexpr int H64_TOTAL = H64_WOUT + HEAD_H + 8;

struct WarpScratch {
    double x[N_INV];              // invariants, then dE/dG
    double y[HEAD_H];             // running activation
    double sd[HEAD_L][HEAD_H];    // SiLU'(pre-activation) per layer
    double dp[HEAD_H];            // dE/dpre of the current layer
    double w[D_ANG * K_RADIAL];   // W_i = dE_i/dP_i (Eq. 7)
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

__global__ void __launch_bounds__(F64_WARPS * 32, 2) k_mega_f64(F64Args k) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    WarpScratch &ws = reinterpret_cast<WarpScratch *>(smem_raw)[wid];
    const int C = k.n_species;
    const int64_t n_warps = (int64_t)gridDim.x * F64_WARPS;
    double e_sum = 0.0, vir[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};
    unsigned long long n_pairs = 0;

    for (int64_t slot = (int64_t)blockIdx.x * F64_WARPS + wid; slot < k.n; slot += n_warps) {
        const int i = k.center_order[slot];
        const double4 pi = k.pos4[i];
        const int si = (int)pi.w;
        const int64_t beg = k.nbr_off[i], end = k.nbr_off[i + 1];
        const double *hd = k.head + (size_t)si * H64_TOTAL;

        // ---------------- Encoding: P = H^T G (Eq. 4), lane = channel ----------------
        double P[D_ANG];
#pragma unroll
        for (int a = 0; a < D_ANG; ++a) P[a] = 0.0;
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
                    for (int a = 0; a < D_ANG; ++a) ws.st[lane][a] = h[a];
#pragma unroll
                    for (int m = 0; m < 4; ++m) ws.st[lane][16 + m] = b[m];
                    const long long off = ((long long)(si * C + (int)pj.w) * (k.knots + 3) + iv) * K_RADIAL;
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
                const double *cf = k.coef + __double_as_longlong(row[20]) + lane;
                double g = row[16] * cf[0];
                g = fma(row[17], cf[K_RADIAL], g);
                g = fma(row[18], cf[2 * K_RADIAL], g);
                g = fma(row[19], cf[3 * K_RADIAL], g);
#pragma unroll
                for (int a = 0; a < D_ANG; ++a) P[a] = fma(row[a], g, P[a]);
            }
            __syncwarp();
        }

        // ---------------- Invariants (Eq. 5, C_l = I) ----------------
        ws.x[lane] = P[0];
        ws.x[32 + lane] = P[1] * P[1] + P[2] * P[2] + P[3] * P[3];
        ws.x[64 + lane] = P[4] * P[4] + P[5] * P[5] + P[6] * P[6] + P[7] * P[7] + P[8] * P[8];
        {
            double s3 = 0.0;
#pragma unroll
            for (int a = 9; a < 16; ++a) s3 = fma(P[a], P[a], s3);
            ws.x[96 + lane] = s3;
        }
        __syncwarp();

        // ---------------- Regression (Eq. 6) and its reverse pass ----------------
        {
            double p0, p1, d0, d1;
            layer_forward<N_INV>(hd + H64_W0T, hd + H64_BIAS, ws.x, lane, p0, p1);
            double y0 = silu_d(p0, d0), y1 = silu_d(p1, d1);
            ws.sd[0][lane] = d0; ws.sd[0][lane + 32] = d1;
            ws.y[lane] = y0; ws.y[lane + 32] = y1;
            __syncwarp();
#pragma unroll 1
            for (int L = 1; L < HEAD_L; ++L) {
                layer_forward<HEAD_H>(hd + H64_WLT + (L - 1) * HEAD_H * HEAD_H, hd + H64_BIAS + L * HEAD_H, ws.y, lane, p0, p1);
                y0 += silu_d(p0, d0); y1 += silu_d(p1, d1);
                __syncwarp();
                ws.sd[L][lane] = d0; ws.sd[L][lane + 32] = d1;
                ws.y[lane] = y0; ws.y[lane + 32] = y1;
                __syncwarp();
            }
            const double wo0 = hd[H64_WOUT + lane], wo1 = hd[H64_WOUT + 32 + lane];
            double e_i = wo0 * y0 + wo1 * y1;
#pragma unroll
            for (int o = 16; o; o >>= 1) e_i += __shfl_xor_sync(0xffffffffu, e_i, o);
            e_i += hd[H64_WOUT + HEAD_H];
            if (lane == 0) { k.e_atom[i] = e_i; e_sum += e_i; }

            // dE/dy of the last layer is w_out; each hidden layer adds W^T (dE/dy . SiLU') through its skip
            double g0 = wo0, g1 = wo1;
#pragma unroll 1
            for (int L = HEAD_L - 1; L >= 1; --L) {
                ws.dp[lane] = g0 * ws.sd[L][lane]; ws.dp[lane + 32] = g1 * ws.sd[L][lane + 32];
                __syncwarp();
                const double *w = hd + H64_WL + (L - 1) * HEAD_H * HEAD_H;
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
            double dx0 = 0.0, dx1 = 0.0, dx2 = 0.0, dx3 = 0.0;   // dE/dG of invariants lane + 32 l
            const double *w0 = hd + H64_W0;
#pragma unroll 4
            for (int o = 0; o < HEAD_H; ++o) {
                const double d = ws.dp[o];
                dx0 = fma(w0[o * N_INV + lane], d, dx0);
                dx1 = fma(w0[o * N_INV + 32 + lane], d, dx1);
                dx2 = fma(w0[o * N_INV + 64 + lane], d, dx2);
                dx3 = fma(w0[o * N_INV + 96 + lane], d, dx3);
            }
            // W_i = dE_i/dP_i (Eq. 7)
            ws.w[lane] = dx0;
#pragma unroll
            for (int a = 1; a < D_ANG; ++a) ws.w[a * K_RADIAL + lane] = 2.0 * (a < 4 ? dx1 : (a < 9 ? dx2 : dx3)) * P[a];
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
                const double *cf = k.coef + ((size_t)(si * C + (int)pj.w) * (k.knots + 3) + iv) * K_RADIAL;
                double v[D_ANG], t[D_ANG];
#pragma unroll
                for (int a = 0; a < D_ANG; ++a) { v[a] = 0.0; t[a] = 0.0; }
#pragma unroll 1
                for (int c = 0; c < K_RADIAL; c += 2) {
                    double g0 = 0.0, g1 = 0.0, dg0 = 0.0, dg1 = 0.0;
#pragma unroll
                    for (int m = 0; m < 4; ++m) {
                        const double2 cc = *reinterpret_cast<const double2 *>(cf + m * K_RADIAL + c);
                        g0 = fma(b[m], cc.x, g0); g1 = fma(b[m], cc.y, g1);
                        dg0 = fma(db[m], cc.x, dg0); dg1 = fma(db[m], cc.y, dg1);
                    }
#pragma unroll
                    for (int a = 0; a < D_ANG; ++a) {
                        const double2 w = *reinterpret_cast<const double2 *>(&ws.w[a * K_RADIAL + c]);
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

// fp64 forces and energies -> the fp32 arrays the fp32 getters and the integrator's fallback read
__global__ void k_force_to_float(int64_t n, const double *__restrict__ fd, const double *__restrict__ ed, float4 *__restrict__ force,
                                 float *__restrict__ e_atom) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    force[i] = make_float4((float)fd[3 * i], (float)fd[3 * i + 1], (float)fd[3 * i + 2], 0.f);
    e_atom[i] = (float)ed[i];
}

int upload_head_f64(mlip_ctx *c, const double *w) {
    const int C = c->cfg.n_species;
    double *host = (double *)calloc((size_t)C * H64_TOTAL, sizeof(double));
    if (!host) return MLIP_ERR_OOM;
    for (int s = 0; s < C; ++s) {
        const double *src = w + (size_t)s * HEAD_NET;
        double *hp = host + (size_t)s * H64_TOTAL;
        int in = N_INV;
        for (int L = 0; L < HEAD_L; ++L) {
            double *row = L == 0 ? hp + H64_W0 : hp + H64_WL + (L - 1) * HEAD_H * HEAD_H;
            double *tr = L == 0 ? hp + H64_W0T : hp + H64_WLT + (L - 1) * HEAD_H * HEAD_H;
            for (int o = 0; o < HEAD_H; ++o)
                for (int q = 0; q < in; ++q) {
                    row[o * in + q] = src[o * in + q];
                    tr[q * HEAD_H + o] = src[o * in + q];
                }
            for (int o = 0; o < HEAD_H; ++o) hp[H64_BIAS + L * HEAD_H + o] = src[in * HEAD_H + o];
            src += in * HEAD_H + HEAD_H;
            in = HEAD_H;
        }
        for (int o = 0; o < HEAD_H + 1; ++o) hp[H64_WOUT + o] = src[o];
    }
    const size_t bytes = sizeof(double) * (size_t)C * H64_TOTAL;
    cudaError_t e = cudaMalloc(&c->head_w_d, bytes);
    if (e == cudaSuccess) e = cudaMemcpy(c->head_w_d, host, bytes, cudaMemcpyHostToDevice);
    free(host);
    if (e != cudaSuccess) { c->err = cudaGetErrorString(e); return MLIP_ERR_CUDA; }
    c->resident += bytes;
    return MLIP_OK;
}

int launch_megakernel_f64(mlip_ctx *c, cudaStream_t s) {
    const int64_t n = c->n;
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->force_d, 0, sizeof(double) * 3 * n, s));
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->acc, 0, sizeof(double) * ACC_KINETIC, s));
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->pair_counter, 0, sizeof(unsigned long long), s));
    const size_t smem_bytes = sizeof(WarpScratch) * F64_WARPS;
    if (!c->kernel_ready) {
        cudaError_t e = cudaFuncSetAttribute(k_mega_f64, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
        if (e != cudaSuccess) { c->err = std::string("fp64 kernel shared memory: ") + cudaGetErrorString(e); return MLIP_ERR_CUDA; }
        c->kernel_ready = true;
    }
    const int blocks = (int)std::min<int64_t>((n + F64_WARPS - 1) / F64_WARPS, (int64_t)2 * c->n_sm);
    F64Args k;
    k.n = n; k.n_species = c->cfg.n_species; k.grid = c->grid; k.rc2 = c->cfg.r_cut * c->cfg.r_cut;
    k.coef = c->table_d; k.knots = c->cfg.table_knots; k.r_min = c->cfg.table_r_min;
    k.inv_h = c->cfg.table_knots / (c->cfg.r_cut - c->cfg.table_r_min);
    k.pos4 = c->pos4; k.center_order = c->center_order; k.nbr_off = c->nbr_off; k.nbr = c->nbr;
    k.head = c->head_w_d; k.force = c->force_d; k.e_atom = c->e_atom_d; k.acc = c->acc;
    k.pair_counter = c->pair_counter; k.status = c->status;
    const int slot = (int)(c->ev_count % mlip_ctx::EV_POOL);
    MLIP_CUDA_TRY(c, cudaEventRecord(c->ev[2 * slot], s));
    k_mega_f64<<<blocks, F64_WARPS * 32, smem_bytes, s>>>(k);
    MLIP_CUDA_TRY(c, cudaEventRecord(c->ev[2 * slot + 1], s));
    c->ev_count += 1;
    k_force_to_float<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(n, c->force_d, c->e_atom_d, c->force, c->e_atom);
    c->launches += 2;
    MLIP_CUDA_TRY(c, cudaGetLastError());
    return MLIP_OK;
}

}  // namespace mlip
