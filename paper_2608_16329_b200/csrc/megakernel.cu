// The fused evaluation kernel (Section 3.4.1 "mega-fusion": Eq. 1-10 in one launch, every
// per-pair and per-atom intermediate kept in registers or shared memory, the radial and
// angular features recomputed in the derivation stage instead of being kept).
//
// Mapping, one warp per central atom:
//   Encoding   lanes = pairs for the geometry (Eq. 1), the harmonics (Eq. 3) and the spline
//              basis; then lanes = radial channels: each lane owns one column of the moment
//              P_i (16 registers) and accumulates h (x) g (Eq. 4) with h broadcast from
//              shared memory.  Invariants (Eq. 5) are then lane-local.
//   Regression the species head (Eq. 6) forward and in reverse, two neurons per lane.
//   Derivation W_i (Eq. 7) goes to shared memory; lanes = pairs again: each lane rebuilds
//              g, g' for its pair, contracts them with W_i (Eq. 9 and the re-associated
//              Eq. 8 term: U_i is never formed), projects onto the pair vector (Eq. 10) and
//              scatters: its own sum stays in registers, the reaction goes out by atomics.
#include "common.cuh"

namespace mlip {

constexpr int WARPS = 8;
constexpr int STAGE_STRIDE = 28;   // floats per lane in the pair -> channel hand-over (16 h, 4 b, offset, pad)

// fp32 head layout per species (floats):
//   forward   W1t[128][64] b1[64] | W2t[64][64] b2[64] | W3t b3 | W4t b4 | w_out[64] b_out pad[3]
//   backward  W1[64][128] | W2[64][64] | W3 | W4      (row-major [out][in], as supplied)
constexpr int HW_FWD = N_INV * HEAD_H + HEAD_H + (HEAD_L - 1) * (HEAD_H * HEAD_H + HEAD_H) + HEAD_H + 4;
constexpr int HW_BWD = N_INV * HEAD_H + (HEAD_L - 1) * HEAD_H * HEAD_H;
constexpr int HW_TOTAL = HW_FWD + HW_BWD;

__device__ __forceinline__ float silu_f(float x, float &dsilu) {
    float s = 1.0f / (1.0f + expf(-x));
    dsilu = s * (1.0f + x * (1.0f - s));
    return x * s;
}

// Irreducible harmonic polynomials up to l = 3 of a unit vector (one valid solution of the
// projection constraints of Section 3.3.1: harmonic, orthonormal under the multinomial metric).
__device__ __forceinline__ void harmonics(float x, float y, float z, float *h) {
    const float s2 = 1.41421356237f, is2 = 0.70710678118f, is6 = 0.40824829046f;
    const float s6 = 2.44948974278f, s15 = 1.22474487139f, is10 = 0.31622776601f;
    float xx = x * x, yy = y * y, zz = z * z;
    h[0] = 1.0f;
    h[1] = x; h[2] = y; h[3] = z;
    h[4] = s2 * x * y; h[5] = s2 * x * z; h[6] = s2 * y * z;
    h[7] = is2 * (xx - yy);
    h[8] = is6 * (2.0f * zz - xx - yy);
    h[9] = s6 * x * y * z;
    h[10] = s15 * z * (xx - yy);
    h[11] = s15 * x * (yy - zz);
    h[12] = s15 * y * (zz - xx);
    h[13] = is10 * x * (2.0f * xx - 3.0f * yy - 3.0f * zz);
    h[14] = is10 * y * (2.0f * yy - 3.0f * xx - 3.0f * zz);
    h[15] = is10 * z * (2.0f * zz - 3.0f * xx - 3.0f * yy);
}

// Accumulate  s += sum_a h_a t_a,  tv += sum_a v_a grad h_a,  tu += sum_a l_a v_a h_a  (Euler: grad h_a . u = l_a h_a).
__device__ __forceinline__ void harmonics_project(float x, float y, float z, const float *v, const float *t,
                                                  float &s, float &tx, float &ty, float &tz, float &tu) {
    const float s2 = 1.41421356237f, is2 = 0.70710678118f, is6 = 0.40824829046f;
    const float s6 = 2.44948974278f, s15 = 1.22474487139f, is10 = 0.31622776601f;
    float xx = x * x, yy = y * y, zz = z * z, h;
    s = t[0]; tx = ty = tz = 0.f; tu = 0.f;
    // l = 1
    s += x * t[1] + y * t[2] + z * t[3];
    tx += v[1]; ty += v[2]; tz += v[3];
    tu += x * v[1] + y * v[2] + z * v[3];
    // l = 2
    float u2 = 0.f;
    h = s2 * x * y; s += h * t[4]; u2 += h * v[4]; tx += s2 * y * v[4]; ty += s2 * x * v[4];
    h = s2 * x * z; s += h * t[5]; u2 += h * v[5]; tx += s2 * z * v[5]; tz += s2 * x * v[5];
    h = s2 * y * z; s += h * t[6]; u2 += h * v[6]; ty += s2 * z * v[6]; tz += s2 * y * v[6];
    h = is2 * (xx - yy); s += h * t[7]; u2 += h * v[7]; tx += s2 * x * v[7]; ty -= s2 * y * v[7];
    h = is6 * (2.f * zz - xx - yy); s += h * t[8]; u2 += h * v[8];
    tx -= 2.f * is6 * x * v[8]; ty -= 2.f * is6 * y * v[8]; tz += 4.f * is6 * z * v[8];
    // l = 3
    float u3 = 0.f;
    h = s6 * x * y * z; s += h * t[9]; u3 += h * v[9];
    tx += s6 * y * z * v[9]; ty += s6 * x * z * v[9]; tz += s6 * x * y * v[9];
    h = s15 * z * (xx - yy); s += h * t[10]; u3 += h * v[10];
    tx += 2.f * s15 * x * z * v[10]; ty -= 2.f * s15 * y * z * v[10]; tz += s15 * (xx - yy) * v[10];
    h = s15 * x * (yy - zz); s += h * t[11]; u3 += h * v[11];
    tx += s15 * (yy - zz) * v[11]; ty += 2.f * s15 * x * y * v[11]; tz -= 2.f * s15 * x * z * v[11];
    h = s15 * y * (zz - xx); s += h * t[12]; u3 += h * v[12];
    tx -= 2.f * s15 * x * y * v[12]; ty += s15 * (zz - xx) * v[12]; tz += 2.f * s15 * y * z * v[12];
    h = is10 * x * (2.f * xx - 3.f * yy - 3.f * zz); s += h * t[13]; u3 += h * v[13];
    tx += is10 * (6.f * xx - 3.f * yy - 3.f * zz) * v[13]; ty -= 6.f * is10 * x * y * v[13]; tz -= 6.f * is10 * x * z * v[13];
    h = is10 * y * (2.f * yy - 3.f * xx - 3.f * zz); s += h * t[14]; u3 += h * v[14];
    tx -= 6.f * is10 * x * y * v[14]; ty += is10 * (6.f * yy - 3.f * xx - 3.f * zz) * v[14]; tz -= 6.f * is10 * y * z * v[14];
    h = is10 * z * (2.f * zz - 3.f * xx - 3.f * yy); s += h * t[15]; u3 += h * v[15];
    tx -= 6.f * is10 * x * z * v[15]; ty -= 6.f * is10 * y * z * v[15]; tz += is10 * (6.f * zz - 3.f * xx - 3.f * yy) * v[15];
    tu += 2.f * u2 + 3.f * u3;
}

struct PairGeom {
    float x, y, z, r, rinv;
    int j;
    bool valid;
};

// Eq. 1 with the periodic minimum image.  Differences are taken in fp64 (positions keep their
// full precision in large boxes) and narrowed afterwards.
__device__ __forceinline__ PairGeom pair_geometry(const double4 &pi, const double4 &pj, const CellGrid &g, double rc2) {
    PairGeom p;
    double dx = min_image(pj.x - pi.x, g.box[0], g.half[0]);
    double dy = min_image(pj.y - pi.y, g.box[1], g.half[1]);
    double dz = min_image(pj.z - pi.z, g.box[2], g.half[2]);
    double d2 = dx * dx + dy * dy + dz * dz;
    p.valid = d2 < rc2;
    p.x = (float)dx; p.y = (float)dy; p.z = (float)dz;
    p.r = sqrtf((float)d2);
    p.rinv = 1.0f / p.r;
    return p;
}

// Spline interval and cubic B-spline basis at distance r.
__device__ __forceinline__ int spline_basis(float r, const TableDesc &tab, float *b, float *db, int *status) {
    float xk = (r - tab.r_min) * tab.inv_h;
    if (xk < 0.f) { atomicOr(status, FLAG_TABLE_RANGE); xk = 0.f; }
    int i = (int)xk;
    i = i > tab.knots - 1 ? tab.knots - 1 : i;
    float u = xk - (float)i, u2 = u * u, u3 = u2 * u, w = 1.f - u;
    const float sixth = 1.0f / 6.0f;
    b[0] = w * w * w * sixth;
    b[1] = (3.f * u3 - 6.f * u2 + 4.f) * sixth;
    b[2] = (-3.f * u3 + 3.f * u2 + 3.f * u + 1.f) * sixth;
    b[3] = u3 * sixth;
    if (db) {
        db[0] = -0.5f * w * w * tab.inv_h;
        db[1] = (1.5f * u2 - 2.f * u) * tab.inv_h;
        db[2] = (-1.5f * u2 + u + 0.5f) * tab.inv_h;
        db[3] = 0.5f * u2 * tab.inv_h;
    }
    return i;
}

__global__ void __launch_bounds__(WARPS * 32) k_mega(int64_t n, int n_species, CellGrid grid, double rc2, TableDesc tab,
                                                     const double4 *__restrict__ pos4, const int32_t *__restrict__ center_order,
                                                     const int64_t *__restrict__ nbr_off, const int32_t *__restrict__ nbr,
                                                     const float *__restrict__ head_w, float4 *__restrict__ force,
                                                     double *__restrict__ acc, unsigned long long *__restrict__ pair_counter,
                                                     int *__restrict__ status) {
    __shared__ __align__(16) float s_stage[WARPS][32 * STAGE_STRIDE];
    __shared__ __align__(16) float s_W[WARPS][D_ANG * K_RADIAL];
    __shared__ __align__(16) float s_x[WARPS][N_INV];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float *stage = s_stage[warp], *sW = s_W[warp], *sx = s_x[warp];
    const int64_t n_warps = (int64_t)gridDim.x * WARPS;
    const int table_rows = tab.knots + 3;

    double e_sum = 0.0;
    float vir[9] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    unsigned long long n_pairs = 0;

    for (int64_t w = (int64_t)blockIdx.x * WARPS + warp; w < n; w += n_warps) {
        const int i = center_order[w];
        const double4 pi = pos4[i];
        const int si = (int)pi.w;
        const int64_t beg = nbr_off[i], end = nbr_off[i + 1];

        // ---------------- Encoding ----------------
        float P[D_ANG];
#pragma unroll
        for (int a = 0; a < D_ANG; ++a) P[a] = 0.f;
        for (int64_t base = beg; base < end; base += 32) {
            const int64_t e = base + lane;
            bool valid = false;
            if (e < end) {
                const int j = nbr[e];
                const double4 pj = pos4[j];
                PairGeom p = pair_geometry(pi, pj, grid, rc2);
                valid = p.valid;
                if (valid) {
                    float h[D_ANG], b[4];
                    harmonics(p.x * p.rinv, p.y * p.rinv, p.z * p.rinv, h);
                    int iv = spline_basis(p.r, tab, b, nullptr, status);
                    int off = ((si * n_species + (int)pj.w) * table_rows + iv) * K_RADIAL;
                    float4 *row = reinterpret_cast<float4 *>(stage + lane * STAGE_STRIDE);
                    row[0] = make_float4(h[0], h[1], h[2], h[3]);
                    row[1] = make_float4(h[4], h[5], h[6], h[7]);
                    row[2] = make_float4(h[8], h[9], h[10], h[11]);
                    row[3] = make_float4(h[12], h[13], h[14], h[15]);
                    row[4] = make_float4(b[0], b[1], b[2], b[3]);
                    row[5] = make_float4(__int_as_float(off), 0.f, 0.f, 0.f);
                }
            }
            unsigned m = __ballot_sync(0xffffffffu, valid);
            n_pairs += __popc(m);
            __syncwarp();
            while (m) {
                const int p = __ffs(m) - 1;
                m &= m - 1;
                const float4 *row = reinterpret_cast<const float4 *>(stage + p * STAGE_STRIDE);
                const float4 b = row[4];
                const int off = __float_as_int(row[5].x);
                const float *tc = tab.coef + off + lane;
                float g = b.x * __ldg(tc) + b.y * __ldg(tc + K_RADIAL) + b.z * __ldg(tc + 2 * K_RADIAL) + b.w * __ldg(tc + 3 * K_RADIAL);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float4 h = row[q];
                    P[4 * q + 0] += h.x * g; P[4 * q + 1] += h.y * g;
                    P[4 * q + 2] += h.z * g; P[4 * q + 3] += h.w * g;
                }
            }
            __syncwarp();
        }

        // ---------------- invariants (Eq. 5, C_l = I) ----------------
        {
            float g1 = P[1] * P[1] + P[2] * P[2] + P[3] * P[3];
            float g2 = P[4] * P[4] + P[5] * P[5] + P[6] * P[6] + P[7] * P[7] + P[8] * P[8];
            float g3 = P[9] * P[9] + P[10] * P[10] + P[11] * P[11] + P[12] * P[12] + P[13] * P[13] + P[14] * P[14] + P[15] * P[15];
            sx[lane] = P[0]; sx[32 + lane] = g1; sx[64 + lane] = g2; sx[96 + lane] = g3;
        }
        __syncwarp();

        // ---------------- Regression (Eq. 6): forward ----------------
        const float *hw = head_w + (size_t)si * HW_TOTAL;
        float dact[HEAD_L][2];   // SiLU'(pre-activation) of this lane's two neurons per layer
        float z0, z1;
        {
            const float *Wt = hw, *bb = hw + N_INV * HEAD_H;
            float a0 = __ldg(bb + lane), a1 = __ldg(bb + 32 + lane);
#pragma unroll 8
            for (int q = 0; q < N_INV; ++q) {
                float x = sx[q];
                a0 += __ldg(Wt + q * HEAD_H + lane) * x;
                a1 += __ldg(Wt + q * HEAD_H + 32 + lane) * x;
            }
            z0 = silu_f(a0, dact[0][0]);
            z1 = silu_f(a1, dact[0][1]);
        }
        const float *layer_w = hw + N_INV * HEAD_H + HEAD_H;
#pragma unroll
        for (int L = 1; L < HEAD_L; ++L) {
            __syncwarp();
            sx[lane] = z0; sx[32 + lane] = z1;
            __syncwarp();
            const float *Wt = layer_w, *bb = layer_w + HEAD_H * HEAD_H;
            float a0 = __ldg(bb + lane), a1 = __ldg(bb + 32 + lane);
#pragma unroll 8
            for (int q = 0; q < HEAD_H; ++q) {
                float x = sx[q];
                a0 += __ldg(Wt + q * HEAD_H + lane) * x;
                a1 += __ldg(Wt + q * HEAD_H + 32 + lane) * x;
            }
            float d0, d1;
            z0 += silu_f(a0, d0);
            z1 += silu_f(a1, d1);
            dact[L][0] = d0; dact[L][1] = d1;
            layer_w += HEAD_H * HEAD_H + HEAD_H;
        }
        const float wo0 = __ldg(layer_w + lane), wo1 = __ldg(layer_w + 32 + lane);
        float e_i = wo0 * z0 + wo1 * z1;
#pragma unroll
        for (int o = 16; o; o >>= 1) e_i += __shfl_xor_sync(0xffffffffu, e_i, o);
        e_i += __ldg(layer_w + HEAD_H);

        // ---------------- Regression in reverse: dE/dG ----------------
        float dz0 = wo0, dz1 = wo1;
        const float *bw = hw + HW_FWD + N_INV * HEAD_H + (HEAD_L - 2) * HEAD_H * HEAD_H;   // W of the last hidden layer
#pragma unroll
        for (int L = HEAD_L - 1; L >= 1; --L) {
            __syncwarp();
            sx[lane] = dz0 * dact[L][0]; sx[32 + lane] = dz1 * dact[L][1];
            __syncwarp();
            float a0 = 0.f, a1 = 0.f;
#pragma unroll 8
            for (int o = 0; o < HEAD_H; ++o) {
                float d = sx[o];
                a0 += __ldg(bw + o * HEAD_H + lane) * d;
                a1 += __ldg(bw + o * HEAD_H + 32 + lane) * d;
            }
            dz0 += a0; dz1 += a1;
            bw -= HEAD_H * HEAD_H;
        }
        __syncwarp();
        sx[lane] = dz0 * dact[0][0]; sx[32 + lane] = dz1 * dact[0][1];
        __syncwarp();
        float dG[4] = {0.f, 0.f, 0.f, 0.f};
        {
            const float *W1 = hw + HW_FWD;
#pragma unroll 4
            for (int o = 0; o < HEAD_H; ++o) {
                float d = sx[o];
#pragma unroll
                for (int q = 0; q < 4; ++q) dG[q] += __ldg(W1 + o * N_INV + 32 * q + lane) * d;
            }
        }

        // ---------------- W_i = dE_i/dP_i (Eq. 7) ----------------
        sW[lane] = dG[0];
#pragma unroll
        for (int a = 1; a < D_ANG; ++a) {
            const float c = 2.0f * (a < 4 ? dG[1] : (a < 9 ? dG[2] : dG[3]));
            sW[a * K_RADIAL + lane] = c * P[a];
        }
        __syncwarp();

        // ---------------- Derivation (Eq. 8-10) ----------------
        float fx = 0.f, fy = 0.f, fz = 0.f;
        for (int64_t base = beg; base < end; base += 32) {
            const int64_t e = base + lane;
            if (e < end) {
                const int j = nbr[e];
                const double4 pj = pos4[j];
                PairGeom p = pair_geometry(pi, pj, grid, rc2);
                if (p.valid) {
                    float b[4], db[4];
                    int iv = spline_basis(p.r, tab, b, db, status);
                    const float4 *tc = reinterpret_cast<const float4 *>(tab.coef + ((si * n_species + (int)pj.w) * table_rows + iv) * K_RADIAL);
                    float v[D_ANG], t[D_ANG];
#pragma unroll
                    for (int a = 0; a < D_ANG; ++a) { v[a] = 0.f; t[a] = 0.f; }
#pragma unroll
                    for (int c4 = 0; c4 < K_RADIAL / 4; ++c4) {
                        float4 c0 = __ldg(tc + c4), c1 = __ldg(tc + 8 + c4), c2 = __ldg(tc + 16 + c4), c3 = __ldg(tc + 24 + c4);
                        float4 g, dg;
                        g.x = b[0] * c0.x + b[1] * c1.x + b[2] * c2.x + b[3] * c3.x;
                        g.y = b[0] * c0.y + b[1] * c1.y + b[2] * c2.y + b[3] * c3.y;
                        g.z = b[0] * c0.z + b[1] * c1.z + b[2] * c2.z + b[3] * c3.z;
                        g.w = b[0] * c0.w + b[1] * c1.w + b[2] * c2.w + b[3] * c3.w;
                        dg.x = db[0] * c0.x + db[1] * c1.x + db[2] * c2.x + db[3] * c3.x;
                        dg.y = db[0] * c0.y + db[1] * c1.y + db[2] * c2.y + db[3] * c3.y;
                        dg.z = db[0] * c0.z + db[1] * c1.z + db[2] * c2.z + db[3] * c3.z;
                        dg.w = db[0] * c0.w + db[1] * c1.w + db[2] * c2.w + db[3] * c3.w;
#pragma unroll
                        for (int a = 0; a < D_ANG; ++a) {
                            const float4 wv = *reinterpret_cast<const float4 *>(sW + a * K_RADIAL + 4 * c4);
                            v[a] += wv.x * g.x + wv.y * g.y + wv.z * g.z + wv.w * g.w;      // Eq. 9: row of V
                            t[a] += wv.x * dg.x + wv.y * dg.y + wv.z * dg.z + wv.w * dg.w;  // W g' (Eq. 8 re-associated)
                        }
                    }
                    const float ux = p.x * p.rinv, uy = p.y * p.rinv, uz = p.z * p.rinv;
                    float s, tx, ty, tz, tu;
                    harmonics_project(ux, uy, uz, v, t, s, tx, ty, tz, tu);
                    // Eq. 10: f_ij = (g' . u_ij) r^ + J_ang^T v_ij,  J_ang = (grad_u h)(I - u u^T) / r
                    const float px = s * ux + (tx - tu * ux) * p.rinv;
                    const float py = s * uy + (ty - tu * uy) * p.rinv;
                    const float pz = s * uz + (tz - tu * uz) * p.rinv;
                    fx += px; fy += py; fz += pz;
                    atomicAdd(&force[j].x, -px);
                    atomicAdd(&force[j].y, -py);
                    atomicAdd(&force[j].z, -pz);
                    vir[0] -= p.x * px; vir[1] -= p.x * py; vir[2] -= p.x * pz;
                    vir[3] -= p.y * px; vir[4] -= p.y * py; vir[5] -= p.y * pz;
                    vir[6] -= p.z * px; vir[7] -= p.z * py; vir[8] -= p.z * pz;
                }
            }
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            fx += __shfl_xor_sync(0xffffffffu, fx, o);
            fy += __shfl_xor_sync(0xffffffffu, fy, o);
            fz += __shfl_xor_sync(0xffffffffu, fz, o);
        }
        if (lane == 0) {
            atomicAdd(&force[i].x, fx);
            atomicAdd(&force[i].y, fy);
            atomicAdd(&force[i].z, fz);
            force[i].w = e_i;
            e_sum += (double)e_i;
        }
        __syncwarp();
    }

    // per-warp totals -> global accumulators
#pragma unroll
    for (int q = 0; q < 9; ++q) {
        float x = vir[q];
#pragma unroll
        for (int o = 16; o; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
        if (lane == 0) atomicAdd(&acc[ACC_VIRIAL + q], (double)x);
    }
    if (lane == 0) {
        atomicAdd(&acc[ACC_ENERGY], e_sum);
        atomicAdd(pair_counter, n_pairs);
    }
}

int upload_head(mlip_ctx *c, const double *w) {
    const int C = c->cfg.n_species;
    std::string buf_err;
    float *host = (float *)malloc(sizeof(float) * (size_t)C * HW_TOTAL);
    if (!host) return MLIP_ERR_OOM;
    for (int s = 0; s < C; ++s) {
        const double *src = w + (size_t)s * HEAD_NET;
        float *fwd = host + (size_t)s * HW_TOTAL, *bwd = fwd + HW_FWD;
        int in = N_INV;
        for (int L = 0; L < HEAD_L; ++L) {
            for (int o = 0; o < HEAD_H; ++o)
                for (int i = 0; i < in; ++i) {
                    fwd[i * HEAD_H + o] = (float)src[o * in + i];
                    bwd[o * in + i] = (float)src[o * in + i];
                }
            for (int o = 0; o < HEAD_H; ++o) fwd[in * HEAD_H + o] = (float)src[in * HEAD_H + o];
            src += in * HEAD_H + HEAD_H;
            fwd += in * HEAD_H + HEAD_H;
            bwd += in * HEAD_H;
            in = HEAD_H;
        }
        for (int o = 0; o < HEAD_H + 1; ++o) fwd[o] = (float)src[o];
        fwd[HEAD_H + 1] = fwd[HEAD_H + 2] = fwd[HEAD_H + 3] = 0.f;
    }
    cudaError_t e = cudaMalloc(&c->head_w, sizeof(float) * (size_t)C * HW_TOTAL);
    if (e == cudaSuccess) e = cudaMemcpy(c->head_w, host, sizeof(float) * (size_t)C * HW_TOTAL, cudaMemcpyHostToDevice);
    free(host);
    if (e != cudaSuccess) { c->err = cudaGetErrorString(e); return MLIP_ERR_CUDA; }
    c->resident += sizeof(float) * (size_t)C * HW_TOTAL;
    return MLIP_OK;
}

int launch_megakernel(mlip_ctx *c, cudaStream_t s) {
    const int64_t n = c->n;
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->force, 0, sizeof(float4) * n, s));
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->acc, 0, sizeof(double) * ACC_KINETIC, s));
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->pair_counter, 0, sizeof(unsigned long long), s));
    int64_t blocks = (n + WARPS - 1) / WARPS;
    const int64_t max_blocks = (int64_t)c->n_sm * 8;
    if (blocks > max_blocks) blocks = max_blocks;
    if (blocks < 1) blocks = 1;
    const double rc2 = c->cfg.r_cut * c->cfg.r_cut;
    const int slot = (int)(c->ev_count % mlip_ctx::EV_POOL);
    MLIP_CUDA_TRY(c, cudaEventRecord(c->ev[2 * slot], s));
    k_mega<<<(unsigned)blocks, WARPS * 32, 0, s>>>(n, c->cfg.n_species, c->grid, rc2, c->tab, c->pos4, c->center_order,
                                                   c->nbr_off, c->nbr, c->head_w, c->force, c->acc, c->pair_counter, c->status);
    MLIP_CUDA_TRY(c, cudaEventRecord(c->ev[2 * slot + 1], s));
    c->ev_count += 1;
    c->launches += 1;
    MLIP_CUDA_TRY(c, cudaGetLastError());
    return MLIP_OK;
}

}  // namespace mlip
