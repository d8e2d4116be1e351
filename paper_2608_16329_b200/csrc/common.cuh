// Internal declarations shared by the library's translation units.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string>

#include "mlip.h"

namespace mlip {

constexpr int K_RADIAL = 32;   // radial channels (Section 3.2.3: k = 32)
constexpr int D_ANG = 16;      // irreducible angular components up to l = 3 (Section 3.3.2)
constexpr int N_INV = 128;     // (l_max + 1) * k invariants (Eq. 5)
constexpr int HEAD_H = 64;     // head width (Section 4.1.3)
constexpr int HEAD_L = 4;      // head hidden layers
constexpr int MAX_SPECIES = 8;
constexpr int MAX_K = 64;      // widest radial feature vector of the fp64 path's shape variants
constexpr size_t head_net_size(int n_inv) {   // doubles per regression network in the caller's layout
    return (size_t)n_inv * HEAD_H + HEAD_H + (size_t)(HEAD_L - 1) * (HEAD_H * HEAD_H + HEAD_H) + HEAD_H + 1;
}
constexpr int HEAD_NET = (int)head_net_size(N_INV);

// 1 eV/(Angstrom amu) in Angstrom/fs^2
constexpr double ACC_UNIT = 1.602176634e-19 / 1.66053906660e-27 * 1e-10;

// device status word bits
enum : int {
    FLAG_NEIGHBOR_OVERFLOW = 1 << 0,
    FLAG_SKIN_EXCEEDED = 1 << 1,
    FLAG_NONFINITE = 1 << 2,
    FLAG_TABLE_RANGE = 1 << 3,
    FLAG_BOUNDS = 1 << 4,   // raised only by builds with -DMLIP_DEBUG_BOUNDS: an index left its array
};

// Range-checked build (-DMLIP_DEBUG_BOUNDS): every index that the fused kernels and the export take from a list or an
// order array is compared with its array's size before it is used; an index out of range raises FLAG_BOUNDS and is
// replaced by 0, so the access still happens inside the array.  Stands in for a memory checker on the kernels' gathers.
#ifdef MLIP_DEBUG_BOUNDS
#define MLIP_CHECK_INDEX(idx, size, status) (((unsigned long long)(idx) < (unsigned long long)(size)) ? (idx) : (atomicOr((status), FLAG_BOUNDS), 0))
#else
#define MLIP_CHECK_INDEX(idx, size, status) (idx)
#endif

// accumulator slots (double)
enum : int { ACC_ENERGY = 0, ACC_VIRIAL = 1, ACC_KINETIC = 10, ACC_COUNT = 32 };
// launch_block in doubles: [0, 4) tile_counter (MAX_SPECIES ints), [4] pair_counter, [5, 15) acc_fx, [16, 16 + ACC_COUNT) acc;
// everything up to the kinetic-energy slot of acc is cleared before every fused-kernel launch
constexpr int LB_PAIR = 4, LB_ACC_FX = 5, LB_ACC = 16, LB_COUNT = LB_ACC + ACC_COUNT;
constexpr size_t LAUNCH_CLEAR_BYTES = sizeof(double) * (LB_ACC + ACC_KINETIC);
static_assert(MAX_SPECIES * sizeof(int) <= LB_PAIR * sizeof(double), "tile counters must fit before the pair counter");

struct CellGrid {
    int n[3];          // cells per dimension
    double inv_edge[3];
    double box[3];
    double half[3];    // 0.5 * box, the minimum-image threshold
    int n_cells;
};

// Radial table: uniform cubic B-spline per ordered species pair and channel.
struct TableDesc {
    const float *coef;   // [C*C][knots + 3][K_RADIAL]
    int knots;           // number of intervals
    float r_min;
    float inv_h;         // 1 / interval width
    float r_cut2;
};

}  // namespace mlip

struct mlip_ctx {
    mlip_config cfg{};
    std::string err;
    int n_sm = 0;

    // model
    float *head_w = nullptr;     // per-species head weights packed in MMA fragment order (megakernel.cu)
    float *table = nullptr;      // spline coefficients
    double *mass = nullptr;      // [C] dev
    double *nhc = nullptr;       // thermostat state {v_eta[3], eta[3], scale, -} (integrate.cu)
    double nhc_nf = 0, nhc_kT = 0, nhc_q1 = 0, nhc_qk = 0;   // parameters of the last NVT call
    // fp64 path (precision = 1) only
    double *head_w_d = nullptr;  // per-species head weights, row-major and transposed (megakernel_f64.cu)
    double *table_d = nullptr;   // spline coefficients in fp64
    double *force_d = nullptr;   // [N][3]
    double *e_atom_d = nullptr;  // [N]
    double table_err_value = 0, table_err_deriv = 0;
    mlip::TableDesc tab{};

    // system (internal order: by cell, then species, then caller index)
    int64_t n = 0, cap_atoms = 0;
    int64_t n_owned = 0;           // atoms that are central atoms (caller indices below it); the rest are ghosts
    mlip::CellGrid grid{};
    int64_t cap_cells = 0;
    double4 *pos4 = nullptr;       // x, y, z, species stored as a double
    double *vel = nullptr;         // [N][3]
    int32_t *user_of = nullptr;    // internal -> caller index
    float4 *force = nullptr;       // fx, fy, fz, unused
    long long *force_fx = nullptr; // [N][3] fixed-point forces, deterministic mode only
    long long *acc_fx = nullptr;   // [10] fixed-point energy and virial, deterministic mode only
    float *e_atom = nullptr;       // E_i, internal order
    float *disp = nullptr;         // [N][3] displacement since the last build
    int32_t *center_order = nullptr;  // internal indices sorted by (species, cell)
    // second set used as the source of a rebuild
    double4 *pos4_src = nullptr;
    double *vel_src = nullptr;
    int32_t *user_src = nullptr;
    // cells
    int32_t *cell_of = nullptr;    // per source atom
    int32_t *cell_count = nullptr, *cell_start = nullptr, *cell_fill = nullptr;   // [n_cells + 1]
    int32_t *bin_count = nullptr, *bin_start = nullptr;                           // [C * n_cells + 1]
    int32_t *species_start = nullptr;  // dev [C + 1]
    // lists
    int32_t *nbr_count = nullptr;  // [N]
    int32_t *nbr_near = nullptr;   // [N] leading entries of each list that were within r_cut + skin / 2 at build time
    int *far_flag = nullptr;       // raised once an atom has moved skin / 4 since the build: the far entries count again
    int64_t *nbr_off = nullptr;    // [N + 1]
    int32_t *nbr = nullptr;        // list entries: int32 indices, or uint16 cell-relative codes when list16
    bool list16 = false;           // format of the current lists (mlip_config.list_format = 1 on a grid of >= 3 cells per edge)
    int32_t *cell_id = nullptr;    // [N] build-time cell of each atom as packed coordinates, internal order (allocated for list_format = 1)
    unsigned long long *tile_state = nullptr;   // [ceil(N / 64) + 1] look-back words of the one-pass rebuild
    int *tile_ticket = nullptr;
    int64_t nbr_cap = 0, n_entries = 0;
    // scratch
    int64_t *scan_tmp = nullptr;   // block sums for the scans
    int64_t scan_tmp_cap = 0;
    double *launch_block = nullptr;   // one allocation: tile_counter, pair_counter, acc_fx, acc back to back, so that a launch
                                      // clears its counters and accumulators with a single memset (LAUNCH_CLEAR_BYTES)
    double *acc = nullptr;         // [ACC_COUNT] (inside launch_block)
    double *kin_part = nullptr;    // [1184] per-block kinetic-energy sums (integrate.cu)
    unsigned long long *pair_counter = nullptr;
    int *status = nullptr;         // device status word
    int *rebuild_flag = nullptr;   // set when an atom has moved beyond the rebuild trigger; pinned copy in rebuild_host
    int *rebuild_host = nullptr;
    int64_t n_builds = 0;
    int lookback_spin_limit = 0;              // polls before a look-back wait of the one-pass list build gives up (0 = default)
    long long lookback_unpublished_tile = -1; // diagnostic list builds only (mlip_debug_rebuild)
    int *tile_counter = nullptr;   // [MAX_SPECIES] dynamic tile scheduler, one counter per central species
    int *status_host = nullptr;    // pinned
    int64_t *total_host = nullptr; // pinned
    double *stage_pos = nullptr;   // [N][3] staging for host entry point
    int32_t *stage_species = nullptr;
    float *stage_force = nullptr;
    double *stage_out = nullptr;   // [10]
    int64_t stage_cap = 0;

    bool built = false, forces_current = false, kernel_ready = false;
    size_t table_bytes = 0;
    int64_t step = 0;
    int64_t launches = 0;
    size_t resident = 0;
    cudaStream_t last_stream = nullptr;
    static constexpr int EV_POOL = 256;
    cudaEvent_t ev[2 * EV_POOL] = {nullptr};
    int64_t ev_count = 0;          // launches timed since the last reset
    // event pairs around list builds and around the integrator's kernels (mlip_get_timings)
    cudaEvent_t ev_build[2 * EV_POOL] = {nullptr}, ev_integrate[2 * EV_POOL] = {nullptr};
    int64_t build_count = 0, integrate_count = 0;
};

namespace mlip {

#define MLIP_CUDA_TRY(ctx, call)                                                          \
    do {                                                                                  \
        cudaError_t e_ = (call);                                                          \
        if (e_ != cudaSuccess) {                                                          \
            (ctx)->err = std::string(#call) + ": " + cudaGetErrorString(e_);              \
            return e_ == cudaErrorMemoryAllocation ? MLIP_ERR_OOM : MLIP_ERR_CUDA;        \
        }                                                                                 \
    } while (0)

// Record the start / stop event of the next slot of a timing pool on stream s.
inline void timing_begin(cudaEvent_t *pool, int64_t count, cudaStream_t s) { cudaEventRecord(pool[2 * (count % mlip_ctx::EV_POOL)], s); }
inline void timing_end(cudaEvent_t *pool, int64_t &count, cudaStream_t s) { cudaEventRecord(pool[2 * (count % mlip_ctx::EV_POOL) + 1], s); count += 1; }

// neighbor.cu
int launch_pack_source(mlip_ctx *c, const double *pos, const int32_t *species, cudaStream_t s);
int launch_build(mlip_ctx *c, bool allow_sync_grow, cudaStream_t s);
int launch_export(mlip_ctx *c, int64_t *seg_ptr, int32_t *nbr, int64_t capacity, int64_t *n_entries_host, cudaStream_t s);
int launch_export_noalloc(mlip_ctx *c, int64_t *seg_ptr, int32_t *nbr, int64_t capacity, int64_t *n_entries_host, cudaStream_t s);
// tables.cu
int build_tables(mlip_ctx *c, const double *enc_w_host, size_t n_enc);
// megakernel.cu
int upload_head(mlip_ctx *c, const double *head_w_host);
int launch_megakernel(mlip_ctx *c, cudaStream_t s);
// megakernel_f64.cu
int upload_head_f64(mlip_ctx *c, const double *head_w_host);
int launch_megakernel_f64(mlip_ctx *c, cudaStream_t s);
bool f64_shape_supported(int k, int l_max, int basis);
// integrate.cu
int launch_kick_drift(mlip_ctx *c, double dt, cudaStream_t s, const double *vscale = nullptr);
int launch_nhc_half(mlip_ctx *c, double n_f, double kT, double q1, double qk, double dt, cudaStream_t s);
int launch_scale_velocities(mlip_ctx *c, cudaStream_t s);
int launch_kick(mlip_ctx *c, double dt, cudaStream_t s);
int launch_kinetic(mlip_ctx *c, cudaStream_t s);
int launch_scatter_forces(mlip_ctx *c, float *forces, float *e_atom, cudaStream_t s);
int launch_scatter_forces_f64(mlip_ctx *c, double *forces, double *e_atom, cudaStream_t s);
int launch_set_positions(mlip_ctx *c, const double *pos, cudaStream_t s);
int launch_set_velocities(mlip_ctx *c, const double *vel, cudaStream_t s);
int launch_get_state(mlip_ctx *c, double *pos, double *vel, cudaStream_t s);

// Compact list entries (neighbor.cu): cell number in the 27-cell traversal order << L16_SHIFT | position inside that cell.
constexpr int L16_SHIFT = 11, L16_MASK = (1 << L16_SHIFT) - 1;
// cell_id[] holds an atom's build-time cell as packed coordinates (10 bits each: no division on the way to the 27 cell
// bases an atom's list needs); grids with more than 1,024 cells along a dimension keep int32 lists.
constexpr int CELL_PACK_BITS = 10, CELL_PACK_MAX = 1 << CELL_PACK_BITS;
__host__ __device__ inline int pack_cell(const CellGrid &g, int linear) {
    const int cz = linear % g.n[2], cy = (linear / g.n[2]) % g.n[1], cx = linear / (g.n[2] * g.n[1]);
    return cx | (cy << CELL_PACK_BITS) | (cz << (2 * CELL_PACK_BITS));
}
__host__ __device__ inline int neighbor_cell(const CellGrid &g, int cid, int it) {
    const int cx = cid & (CELL_PACK_MAX - 1), cy = (cid >> CELL_PACK_BITS) & (CELL_PACK_MAX - 1), cz = cid >> (2 * CELL_PACK_BITS);
    int x = cx + it / 9 - 1, y = cy + (it / 3) % 3 - 1, z = cz + it % 3 - 1;
    x = x < 0 ? x + g.n[0] : (x >= g.n[0] ? x - g.n[0] : x);
    y = y < 0 ? y + g.n[1] : (y >= g.n[1] ? y - g.n[1] : y);
    z = z < 0 ? z + g.n[2] : (z >= g.n[2] ? z - g.n[2] : z);
    return (x * g.n[1] + y) * g.n[2] + z;
}

// Exact minimum-image squared distance in fp64, every operation rounded on its own
// (no fused multiply-add), identical on host and device.
__device__ __forceinline__ double min_image(double d, double box, double half) {
    if (d > half) d = __dsub_rn(d, box);
    else if (d < -half) d = __dadd_rn(d, box);
    return d;
}

// Optional per-phase cycle counters (profiling builds only: -DMLIP_PHASE_CLOCKS).  Slots 16.. of
// the accumulator array receive the summed clock64 ticks of lane 0 of every warp.
#ifdef MLIP_PHASE_CLOCKS
struct PhaseClock {
    long long t, acc[16];
    __device__ __forceinline__ void start() { t = clock64(); for (int q = 0; q < 16; ++q) acc[q] = 0; }
    __device__ __forceinline__ void mark(int slot) { const long long now = clock64(); acc[slot] += now - t; t = now; }
    __device__ __forceinline__ void flush(double *a, int lane) { if (lane == 0) for (int q = 0; q < 16; ++q) atomicAdd(&a[16 + q], (double)acc[q]); }
};
#else
struct PhaseClock {
    __device__ __forceinline__ void start() {}
    __device__ __forceinline__ void mark(int) {}
    __device__ __forceinline__ void flush(double *, int) {}
};
#endif

}  // namespace mlip
