// Velocity-Verlet NVE pieces and the permutation kernels between the caller's atom
// order and the internal cell-sorted order.  Positions and velocities are fp64: at 8 M atoms
// the box is ~450 Angstrom and a 1 fs displacement (~1e-3 Angstrom) would lose most of its
// digits in fp32.
#include "common.cuh"

namespace mlip {

// Force on atom i: the fp64 array when the context evaluates in fp64, else the fp32 one.
__device__ __forceinline__ double3 load_force(const float4 *__restrict__ force, const double *__restrict__ force_d, int64_t i) {
    if (force_d) return make_double3(force_d[3 * i], force_d[3 * i + 1], force_d[3 * i + 2]);
    const float4 f = force[i];
    return make_double3(f.x, f.y, f.z);
}

// v += dt/2 a;  x += dt v;  wrap into [0, L);  track the displacement since the last list build.
__global__ void k_kick_drift(int64_t n, double dt, CellGrid g, const double *__restrict__ mass, float skin_half2,
                             double4 *__restrict__ pos4, double *__restrict__ vel, const float4 *__restrict__ force,
                             const double *__restrict__ force_d, float *__restrict__ disp, int *status, float trigger2,
                             int *rebuild_flag, const double *__restrict__ vscale, float far2, int *far_flag) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    double4 p = pos4[i];
    const double3 f = load_force(force, force_d, i);
    const double k = 0.5 * dt * ACC_UNIT / mass[(int)p.w];
    const double sc = vscale ? *vscale : 1.0;   // thermostat factor applied ahead of the kick (NVT)
    double v[3] = {vel[3 * i] * sc + k * f.x, vel[3 * i + 1] * sc + k * f.y, vel[3 * i + 2] * sc + k * f.z};
    double x[3] = {p.x + dt * v[0], p.y + dt * v[1], p.z + dt * v[2]};
    float d2 = 0.f;
#pragma unroll
    for (int a = 0; a < 3; ++a) {
        vel[3 * i + a] = v[a];
        float d = disp[3 * i + a] + (float)(dt * v[a]);
        disp[3 * i + a] = d;
        d2 += d * d;
        const double L = g.box[a];
        if (x[a] >= L) x[a] -= L;
        else if (x[a] < 0.0) x[a] += L;
        if (!(x[a] >= 0.0 && x[a] < L)) x[a] = 0.0;   // -eps + L rounds to L; NaN is reported below
    }
    if (!(d2 <= skin_half2)) atomicOr(status, d2 == d2 ? FLAG_SKIN_EXCEEDED : FLAG_NONFINITE);
    if (d2 > trigger2) *rebuild_flag = 1;   // same value from every writer
    if (!(d2 <= far2)) *far_flag = 1;       // from now on the lists' far entries may come inside r_cut
    pos4[i] = make_double4(x[0], x[1], x[2], p.w);
}

// v += dt/2 a
__global__ void k_kick(int64_t n, double dt, const double *__restrict__ mass, const double4 *__restrict__ pos4,
                       double *__restrict__ vel, const float4 *__restrict__ force, const double *__restrict__ force_d) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const double3 f = load_force(force, force_d, i);
    const double k = 0.5 * dt * ACC_UNIT / mass[(int)pos4[i].w];
    vel[3 * i] += k * f.x; vel[3 * i + 1] += k * f.y; vel[3 * i + 2] += k * f.z;
}

// Half-step (dt/2) of a Nose-Hoover chain of three thermostats coupled to the kinetic energy in acc[ACC_KINETIC]
// (Martyna-Tuckerman-Tobias-Klein factorisation, one Suzuki-Yoshida term).  One thread.  state = {v_eta[3], eta[3], scale}:
//   dv_eta_k/dt = G_k - v_eta_{k+1} v_eta_k,  G_1 = (2 KE - N_f kT) / Q_1,  G_k = (Q_{k-1} v_eta_{k-1}^2 - kT) / Q_k,
//   particle velocities scale by exp(-v_eta_1 dt/2); the stored kinetic energy is scaled with them.
__global__ void k_nhc_half(double *state, double *acc, double n_f, double kT, double q1, double qk, double dt) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    constexpr int M = 3;
    double v[M] = {state[0], state[1], state[2]};
    const double q[M] = {q1, qk, qk}, d = 0.5 * dt;
    double ke2 = 2.0 * acc[ACC_KINETIC];
    double G[M];
    G[0] = (ke2 - n_f * kT) / q[0];
    for (int c = 1; c < M; ++c) G[c] = (q[c - 1] * v[c - 1] * v[c - 1] - kT) / q[c];
    v[M - 1] += 0.5 * d * G[M - 1];
    for (int c = M - 2; c >= 0; --c) {
        const double a = exp(-0.25 * d * v[c + 1]);
        v[c] = (v[c] * a + 0.5 * d * G[c]) * a;
    }
    const double scale = exp(-d * v[0]);
    ke2 *= scale * scale;
    for (int c = 0; c < M; ++c) state[3 + c] += d * v[c];
    G[0] = (ke2 - n_f * kT) / q[0];
    for (int c = 0; c < M - 1; ++c) {
        const double a = exp(-0.25 * d * v[c + 1]);
        v[c] = (v[c] * a + 0.5 * d * G[c]) * a;
        G[c + 1] = (q[c] * v[c] * v[c] - kT) / q[c + 1];
    }
    v[M - 1] += 0.5 * d * G[M - 1];
    for (int c = 0; c < M; ++c) state[c] = v[c];
    state[6] = scale;
    acc[ACC_KINETIC] = 0.5 * ke2;
}

__global__ void k_scale_velocities(int64_t n3, double *__restrict__ vel, const double *__restrict__ scale) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n3) vel[i] *= *scale;
}

// Kinetic energy in two steps with a fixed summation order (grid-stride partial sums per block, then one warp adds the
// block sums in index order), so that the thermostat -- and with it an NVT trajectory -- is bit-reproducible.
constexpr int KIN_BLOCKS = 1184;
__global__ void k_kinetic(int64_t n, const double *__restrict__ mass, const double4 *__restrict__ pos4,
                          const double *__restrict__ vel, double *__restrict__ block_sum) {
    __shared__ double part[32];
    double e = 0.0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        double vx = vel[3 * i], vy = vel[3 * i + 1], vz = vel[3 * i + 2];
        e += 0.5 * mass[(int)pos4[i].w] * (vx * vx + vy * vy + vz * vz);
    }
    for (int o = 16; o; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = e;
    __syncthreads();
    if (threadIdx.x < 32) {
        e = threadIdx.x < (blockDim.x >> 5) ? part[threadIdx.x] : 0.0;
        for (int o = 16; o; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
        if (threadIdx.x == 0) block_sum[blockIdx.x] = e;
    }
}
__global__ void k_kinetic_finish(int n_blocks, const double *__restrict__ block_sum, double *acc) {
    double e = 0.0;
    for (int b = threadIdx.x; b < n_blocks; b += 32) e += block_sum[b];
    for (int o = 16; o; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
    if (threadIdx.x == 0) acc[ACC_KINETIC] = e / ACC_UNIT;
}

__global__ void k_scatter_forces(int64_t n, const int32_t *__restrict__ user_of, const float4 *__restrict__ force,
                                 const float *__restrict__ e_in, float *__restrict__ forces_out, float *__restrict__ e_atom) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const float4 f = force[i];
    const int64_t u = user_of[i];
    if (forces_out) { forces_out[3 * u] = f.x; forces_out[3 * u + 1] = f.y; forces_out[3 * u + 2] = f.z; }
    if (e_atom) e_atom[u] = e_in[i];
}

__global__ void k_scatter_forces_f64(int64_t n, const int32_t *__restrict__ user_of, const double *__restrict__ force,
                                     const double *__restrict__ e_in, double *__restrict__ forces_out, double *__restrict__ e_atom) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int64_t u = user_of[i];
    if (forces_out) { forces_out[3 * u] = force[3 * i]; forces_out[3 * u + 1] = force[3 * i + 1]; forces_out[3 * u + 2] = force[3 * i + 2]; }
    if (e_atom) e_atom[u] = e_in[i];
}

__global__ void k_set_positions(int64_t n, const int32_t *__restrict__ user_of, const double *__restrict__ pos,
                                CellGrid g, float skin_half2, double4 *__restrict__ pos4, float *__restrict__ disp, int *status,
                                float far2, int *far_flag) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int64_t u = user_of[i];
    double4 p = pos4[i];
    const double x[3] = {pos[3 * u], pos[3 * u + 1], pos[3 * u + 2]};
    const double old[3] = {p.x, p.y, p.z};
    float d2 = 0.f;
    bool ok = true;
#pragma unroll
    for (int a = 0; a < 3; ++a) {
        ok = ok && (x[a] >= 0.0 && x[a] < g.box[a]);
        float d = disp[3 * i + a] + (float)min_image(x[a] - old[a], g.box[a], g.half[a]);
        disp[3 * i + a] = d;
        d2 += d * d;
    }
    if (!ok) atomicOr(status, FLAG_NONFINITE);
    else if (!(d2 <= skin_half2)) atomicOr(status, FLAG_SKIN_EXCEEDED);
    if (!(d2 <= far2)) *far_flag = 1;
    pos4[i] = make_double4(x[0], x[1], x[2], p.w);
}

__global__ void k_set_velocities(int64_t n, const int32_t *__restrict__ user_of, const double *__restrict__ vel_in,
                                 double *__restrict__ vel) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int64_t u = user_of[i];
    vel[3 * i] = vel_in[3 * u]; vel[3 * i + 1] = vel_in[3 * u + 1]; vel[3 * i + 2] = vel_in[3 * u + 2];
}

__global__ void k_get_state(int64_t n, const int32_t *__restrict__ user_of, const double4 *__restrict__ pos4,
                            const double *__restrict__ vel, double *__restrict__ pos_out, double *__restrict__ vel_out) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int64_t u = user_of[i];
    if (pos_out) { double4 p = pos4[i]; pos_out[3 * u] = p.x; pos_out[3 * u + 1] = p.y; pos_out[3 * u + 2] = p.z; }
    if (vel_out) { vel_out[3 * u] = vel[3 * i]; vel_out[3 * u + 1] = vel[3 * i + 1]; vel_out[3 * u + 2] = vel[3 * i + 2]; }
}

static inline unsigned nb(int64_t n) { return (unsigned)((n + 255) / 256); }
static inline float skin_half2(const mlip_ctx *c) { float h = 0.5f * (float)c->cfg.skin; return h * h; }
// Far entries lie beyond r_cut + skin / 2 at build time; a pair closes by at most twice the largest displacement, so they
// stay outside r_cut while every atom has moved less than skin / 4 (0.245: room for the fp32 bookkeeping).
static inline float far_trigger2(const mlip_ctx *c) { float h = 0.245f * (float)c->cfg.skin; return h * h; }

int launch_kick_drift(mlip_ctx *c, double dt, cudaStream_t s, const double *vscale) {
    timing_begin(c->ev_integrate, c->integrate_count, s);
    k_kick_drift<<<nb(c->n), 256, 0, s>>>(c->n, dt, c->grid, c->mass, skin_half2(c), c->pos4, c->vel, c->force, c->force_d, c->disp, c->status,
                                               0.64f * skin_half2(c), c->rebuild_flag, vscale, far_trigger2(c), c->far_flag);
    timing_end(c->ev_integrate, c->integrate_count, s);
    c->launches += 1;
    MLIP_CUDA_TRY(c, cudaGetLastError());
    return MLIP_OK;
}
int launch_kick(mlip_ctx *c, double dt, cudaStream_t s) {
    timing_begin(c->ev_integrate, c->integrate_count, s);
    k_kick<<<nb(c->n), 256, 0, s>>>(c->n, dt, c->mass, c->pos4, c->vel, c->force, c->force_d);
    timing_end(c->ev_integrate, c->integrate_count, s);
    c->launches += 1;
    MLIP_CUDA_TRY(c, cudaGetLastError());
    return MLIP_OK;
}
int launch_nhc_half(mlip_ctx *c, double n_f, double kT, double q1, double qk, double dt, cudaStream_t s) {
    timing_begin(c->ev_integrate, c->integrate_count, s);
    k_nhc_half<<<1, 32, 0, s>>>(c->nhc, c->acc, n_f, kT, q1, qk, dt);
    timing_end(c->ev_integrate, c->integrate_count, s);
    c->launches += 1;
    MLIP_CUDA_TRY(c, cudaGetLastError());
    return MLIP_OK;
}
int launch_scale_velocities(mlip_ctx *c, cudaStream_t s) {
    timing_begin(c->ev_integrate, c->integrate_count, s);
    k_scale_velocities<<<nb(3 * c->n), 256, 0, s>>>(3 * c->n, c->vel, c->nhc + 6);
    timing_end(c->ev_integrate, c->integrate_count, s);
    c->launches += 1;
    MLIP_CUDA_TRY(c, cudaGetLastError());
    return MLIP_OK;
}
int launch_kinetic(mlip_ctx *c, cudaStream_t s) {
    int64_t blocks = nb(c->n);
    if (blocks > KIN_BLOCKS) blocks = KIN_BLOCKS;
    k_kinetic<<<(unsigned)blocks, 256, 0, s>>>(c->n, c->mass, c->pos4, c->vel, c->kin_part);
    k_kinetic_finish<<<1, 32, 0, s>>>((int)blocks, c->kin_part, c->acc);
    c->launches += 2;
    MLIP_CUDA_TRY(c, cudaGetLastError());
    return MLIP_OK;
}
int launch_scatter_forces(mlip_ctx *c, float *forces, float *e_atom, cudaStream_t s) {
    k_scatter_forces<<<nb(c->n), 256, 0, s>>>(c->n, c->user_of, c->force, c->e_atom, forces, e_atom);
    c->launches += 1;
    MLIP_CUDA_TRY(c, cudaGetLastError());
    return MLIP_OK;
}
int launch_scatter_forces_f64(mlip_ctx *c, double *forces, double *e_atom, cudaStream_t s) {
    k_scatter_forces_f64<<<nb(c->n), 256, 0, s>>>(c->n, c->user_of, c->force_d, c->e_atom_d, forces, e_atom);
    c->launches += 1;
    MLIP_CUDA_TRY(c, cudaGetLastError());
    return MLIP_OK;
}
int launch_set_positions(mlip_ctx *c, const double *pos, cudaStream_t s) {
    k_set_positions<<<nb(c->n), 256, 0, s>>>(c->n, c->user_of, pos, c->grid, skin_half2(c), c->pos4, c->disp, c->status, far_trigger2(c), c->far_flag);
    c->launches += 1;
    MLIP_CUDA_TRY(c, cudaGetLastError());
    return MLIP_OK;
}
int launch_set_velocities(mlip_ctx *c, const double *vel, cudaStream_t s) {
    k_set_velocities<<<nb(c->n), 256, 0, s>>>(c->n, c->user_of, vel, c->vel);
    c->launches += 1;
    MLIP_CUDA_TRY(c, cudaGetLastError());
    return MLIP_OK;
}
int launch_get_state(mlip_ctx *c, double *pos, double *vel, cudaStream_t s) {
    k_get_state<<<nb(c->n), 256, 0, s>>>(c->n, c->user_of, c->pos4, c->vel, pos, vel);
    c->launches += 1;
    MLIP_CUDA_TRY(c, cudaGetLastError());
    return MLIP_OK;
}

}  // namespace mlip
