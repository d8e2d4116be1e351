/*
 * mlip.h - C ABI of the B200 (sm_100a) small-footprint MLIP library.
 *
 * The library evaluates per-atom energies, forces and the virial of the
 * pair-conditioned, irreducible-angular-basis potential (paper Section 3.1,
 * Eq. 1-10) for periodic orthorhombic multi-component systems: a cell-binned
 * neighbor list followed by ONE fused kernel (Section 3.4, "mega-fusion") that
 * runs encoding, regression and derivation without writing a feature vector or
 * any per-pair / per-atom intermediate tensor to device memory; plus a
 * velocity-Verlet NVE step around it.
 *
 * Conventions
 *   - Every function returns an int status (MLIP_OK == 0).  Nothing throws or
 *     aborts, and no kernel traps: a device-side problem (list capacity, skin
 *     exceeded, non-finite input, distance below the table range) raises a bit
 *     in a device status word, the kernels finish with defined output, and the
 *     next mlip_sync_status() reports and clears it.
 *   - "dev" pointers are device memory on the context's device, "host" pointers
 *     are host memory.  The caller owns every buffer it passes; the library
 *     owns the context and its internal buffers until mlip_destroy().
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls enqueue work and return without synchronising unless stated.
 *   - Units: Angstrom, eV, amu, fs.  Atom order of every array argument is the
 *     caller's; the library keeps its own cell-sorted order internally.
 *   - The fp32 path is compiled for k = 32 radial channels and l_max = 3 (d = 16), the paper's production
 *     shape; models with k < 32 or l_max < 3 run in it unchanged in value (their missing channels and orders are
 *     zero-filled at create time) but at the full shape's cost; the fp64 path (precision = 1) also for k in {16, 32, 64} x l_max in {1, 2, 3}, for k = 32 with
 *     l_max = 4, 5 (d = 25, 36), and for the canonical angular basis (config.basis = 1) with k in {32, 64}.  The
 *     encoder is 1 -> enc_hidden x enc_layers -> k, the head is
 *     (l_max+1) k -> head_hidden x head_layers -> 1 with head_hidden = 64,
 *     head_layers = 4 (Section 4.1.3), SiLU, identity skips around hidden
 *     layers of equal width.
 */
#ifndef MLIP_H
#define MLIP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mlip_ctx mlip_ctx;

enum {
    MLIP_OK = 0,
    MLIP_ERR_INVALID_ARG = 1,
    MLIP_ERR_UNSUPPORTED = 2,      /* k, l_max, network shape, species count not compiled in */
    MLIP_ERR_BOX_TOO_SMALL = 3,    /* an edge is shorter than 2 (r_cut + skin) */
    MLIP_ERR_NEIGHBOR_OVERFLOW = 4,/* list capacity exceeded during an in-step rebuild (the fused kernel then skips its
                                      evaluations until the lists are rebuilt by mlip_build_neighbors) */
    MLIP_ERR_SKIN_EXCEEDED = 5,    /* an atom moved more than skin/2 since the last build */
    MLIP_ERR_NONFINITE = 6,        /* NaN/Inf or out-of-box position, species out of range, over-full cell */
    MLIP_ERR_TABLE_TOLERANCE = 7,  /* radial table misses the encoder by more than table_tol */
    MLIP_ERR_NOT_BUILT = 8,        /* compute/step before build_neighbors */
    MLIP_ERR_OOM = 9,
    MLIP_ERR_CUDA = 10,
    MLIP_ERR_TABLE_RANGE = 11      /* a pair came closer than table_r_min */
};

typedef struct {
    int n_species;        /* C, 1..8 */
    double r_cut;         /* Angstrom */
    double skin;          /* list radius = r_cut + skin */
    int k;                /* 1 .. 32 (precision 1: 16, 32 or 64) */
    int l_max;            /* 0 .. 3 (precision 1: 1 .. 5, see above) */
    int enc_hidden, enc_layers;    /* e.g. 128, 3 */
    int head_hidden, head_layers;  /* 64, 4 */
    int table_knots;      /* intervals of the radial table on [table_r_min, r_cut]; 0 = automatic: 64, doubled until table_tol holds */
    double table_r_min;   /* smallest tabulated distance; 0 = default (1.0) */
    double table_tol;     /* accepted table error relative to max|g|; 0 = default (1e-6; with precision 1: 1e-10, and 100 x that for g') */
    int device;           /* CUDA device ordinal */
    int precision;        /* 0: fp32 with the contractions on the tensor pipe (split TF32), the production path;
                             1: every step of Eq. 1-10 in fp64 (Section 4.2 evaluates in double precision by default):
                                fp64 tables (automatic knots start at 512), fp64 forces kept for the integrator,
                                +32 bytes per atom, several times slower */
    int enc_conditioning; /* species information given to the encoder (Section 3.2.2): 0 = the pair (s_i, s_j), C*C nets
                             (the paper's choice); 1 = the neighbor species s_j, C nets; 2 = none, one net */
    int head_conditioning;/* ... to the regression network: 0 = central species s_i, C nets; 1 = none, one net */
    int force_mode;       /* 0: floating-point atomics for the force scatter and the energy / virial totals (results vary in
                             the last bits from run to run); 1: deterministic -- those sums are taken in integer arithmetic
                             (forces in units of 2^-32 eV/Angstrom), so equal inputs give bit-identical outputs and
                             trajectories, NVE and NVT alike (the thermostat's kinetic energy is summed in a fixed order in
                             either mode); +24 bytes per atom, fp32 path only */
    int envelope;         /* smooth cutoff f_c multiplying the encoder output (the paper names none): 0 = (1 + cos(pi r / r_c)) / 2,
                             1 = 1 - 10 x^3 + 15 x^4 - 6 x^5 with x = r / r_c (second derivative also vanishes at r_c) */
    int basis;            /* angular basis (Section 3.3): 0 = irreducible harmonics, d = (l_max + 1)^2, C_l = I (the paper's
                             choice); 1 = canonical: every Cartesian monomial of the unit vector up to degree l_max,
                             d = 4, 10, 20 for l_max = 1, 2, 3 (Eq. 11), with C_l = the multinomial multiplicities in Eq. 5
                             -- the descriptor "before reduction" of Table 7; precision 1 only */
    int list_format;      /* storage of the neighbor lists, the bulk of the footprint (Section 1 and Fig. 4(b): atoms per GPU
                             are bounded by memory): 0 = int32 indices, 4 bytes per entry; 1 = 16-bit codes (which of the 27
                             cells around the atom's own cell, position inside it), 2 bytes per entry + 4 per atom, decoded
                             inside the kernels; same lists, same results.  Falls back to format 0 on grids with fewer
                             than three cells along an edge */
} mlip_config;

/*
 * Create a context: uploads the networks, tabulates every ordered-pair encoder
 * (Eq. 2: g = f_c(r) E(r; s_i, s_j), cosine envelope f_c) as a cubic B-spline
 * in fp64 on the device and checks it against the network.  Synchronises.
 *   enc_weights_host  [C*C] nets, net index s_i*C + s_j ([C] nets indexed s_j, or one net, with
 *                     enc_conditioning 1 or 2); each net is
 *                     W1[h][1], b1[h], W2[h][h], b2[h], ..., Wout[k][h], bout[k], row-major [out][in]
 *   head_weights_host [C] nets (one with head_conditioning 1); each W1[64][128], b1, W2[64][64], b2, ..., w_out[64], b_out
 *   mass_amu_host     [C]
 * Errors: INVALID_ARG, UNSUPPORTED, OOM, CUDA, TABLE_TOLERANCE (context is still returned
 * for inspection through mlip_table_error when the tolerance fails, *out otherwise NULL).
 */
int mlip_create(mlip_ctx **out, const mlip_config *cfg,
                const double *enc_weights_host, size_t n_enc,
                const double *head_weights_host, size_t n_head,
                const double *mass_amu_host);

/* Largest |spline - network| / max|network| found over all pair types (value, derivative). */
int mlip_table_error(const mlip_ctx *ctx, double *err_value, double *err_deriv);

/*
 * Bin the atoms into cells and build the neighbor lists (Section 3.1.1: all j
 * within the list radius, minimum image, strict d^2 < (r_cut+skin)^2 in fp64
 * without fused multiply-add).  Copies positions and species into the context;
 * velocities are reset to zero.  Positions must lie in [0, L).  May reallocate
 * and synchronises once (to size the list).
 *   pos      dev [N][3] double      species  dev [N] int32 in [0, C)
 *   box      host [9]: the three cell vectors, row-major (a_x a_y a_z  b_x b_y b_z  c_x c_y c_z).  Only orthorhombic
 *            cells aligned with the axes are compiled in: a non-zero off-diagonal entry gives MLIP_ERR_UNSUPPORTED;
 *            each edge (the diagonal) must be >= 2 (r_cut + skin), else MLIP_ERR_BOX_TOO_SMALL.
 * A non-finite or out-of-box position, a species outside [0, C) or more than 1,024 atoms in one cell is reported at once
 * as MLIP_ERR_NONFINITE (no lists are built).
 */
int mlip_build_neighbors(mlip_ctx *ctx, int64_t n_atoms, const double *pos, const int32_t *species,
                         const double *box, void *stream);

/*
 * The same build for one sub-domain of a spatial decomposition (Section 3.5 couples the potential to an MD code that
 * decomposes space and exchanges ghost atoms over MPI; Section 4.4 scales it that way).  The first n_owned atoms are this
 * domain's own: they are the central atoms i of Eq. 4-10.  The n_ghost atoms after them are copies of other domains'
 * atoms within r_cut + skin of the domain: they appear as neighbors j only -- no list, no E_i of their own.
 *   pos / species   dev [n_owned + n_ghost], owned atoms first
 *   box             as above.  In a dimension that is split, give the sub-domain's extent including its halos plus at
 *                   least r_cut + skin of empty space, with coordinates shifted into [0, L): the periodic image across
 *                   the padding is then out of reach and the dimension behaves as open.
 * mlip_compute then returns, in the caller's order, the forces its central atoms exert: on owned atoms the part of
 * F_a that comes from this domain's E_i, on the ghosts (entries n_owned ..) the reaction forces -dE_i/dr_a that the
 * caller must send back to the ghosts' owners and add there.  Energy and virial are this domain's central atoms' sums;
 * e_atom of a ghost is 0.  Summed over domains the results equal the single-domain evaluation.  New ghost positions
 * arrive through mlip_set_positions; mlip_step and mlip_step_nvt return MLIP_ERR_UNSUPPORTED on such a context.
 */
int mlip_build_neighbors_ghost(mlip_ctx *ctx, int64_t n_owned, int64_t n_ghost, const double *pos, const int32_t *species,
                               const double *box, void *stream);

/*
 * Export the lists in canonical form: caller's atom indices; for atom i and
 * species s the neighbors of species s in ascending index order occupy
 * nbr[seg_ptr[i*C+s] .. seg_ptr[i*C+s+1]).  Synchronises.
 *   seg_ptr dev [N*C+1] int64, nbr dev [capacity] int32, n_entries_host out.
 * If capacity is too small only seg_ptr and *n_entries_host are valid and
 * MLIP_ERR_NEIGHBOR_OVERFLOW is returned.  While the status word holds a list overflow or a broken configuration from
 * an in-step rebuild (see mlip_sync_status) the lists are incomplete and the call returns that error without exporting.
 */
int mlip_get_neighbors(mlip_ctx *ctx, int64_t *seg_ptr, int32_t *nbr, int64_t capacity,
                       int64_t *n_entries_host, void *stream);

/*
 * mlip_get_neighbors without any allocation (the paper has no counterpart: this is a
 * deployment variant, not a step of its method).  Same arguments, same output, same status codes.
 * mlip_get_neighbors takes two temporary device blocks with cudaMalloc on every call; some callers
 * cannot afford that: an MD driver that has handed all device memory to its own pools, a plug-in
 * that must not disturb its host's allocator, code running where an allocation would stall every
 * stream.  This variant keeps those temporaries in a static device array of about 4 MiB that every
 * GPU loading the library holds until the process exits, and calls no cudaMalloc, cudaFree or
 * allocating library routine.
 *   Limit: n_atoms * n_species <= 1,048,576; larger systems get MLIP_ERR_UNSUPPORTED.
 *   The first call on a device looks up the array's device address (once per device, with that
 *   device current); make that first call before starting any stream capture.
 *   All calls share the array and it keeps the previous call's contents (every word that is read
 *   is rewritten first, so nothing needs clearing); calls whose kernels overlap on one GPU race on
 *   it - issue them one after another.
 * Synchronises, like mlip_get_neighbors.
 */
int mlip_get_neighbors_noalloc(mlip_ctx *ctx, int64_t *seg_ptr, int32_t *nbr, int64_t capacity,
                               int64_t *n_entries_host, void *stream);

/* Replace positions (dev [N][3], caller's order) keeping the current lists. */
int mlip_set_positions(mlip_ctx *ctx, const double *pos, void *stream);
/* Set velocities (dev [N][3], Angstrom/fs, caller's order). */
int mlip_set_velocities(mlip_ctx *ctx, const double *vel, void *stream);

/*
 * One fused evaluation (Eq. 1-10) at the current positions with the current
 * lists.  Any output pointer may be NULL.
 *   energy dev [1] double (sum of E_i)      forces dev [N][3] float, F = -dE/dr
 *   virial dev [9] double, row-major Xi_ab = -sum_i sum_j (r_ij)_a (dE_i/dr_ij)_b
 *   e_atom dev [N] float
 */
int mlip_compute(mlip_ctx *ctx, double *energy, float *forces, double *virial, float *e_atom, void *stream);

/*
 * The same evaluation with fp64 per-atom outputs (forces dev [N][3] double,
 * e_atom dev [N] double), for contexts created with precision = 1; returns
 * MLIP_ERR_UNSUPPORTED on an fp32 context.  mlip_compute() on an fp64 context
 * runs the fp64 kernel and rounds the per-atom outputs to float.
 */
int mlip_compute_f64(mlip_ctx *ctx, double *energy, double *forces, double *virial, double *e_atom, void *stream);

/*
 * Same evaluation with HOST buffers: copies positions in (and species at a
 * rebuild), rebuilds the lists when `rebuild` != 0 or none exist, evaluates,
 * copies results out and synchronises.  This is the call a host-side MD code
 * makes once per time step.  box_host as in mlip_build_neighbors ([9], row-major cell vectors).
 */
int mlip_compute_host(mlip_ctx *ctx, int64_t n_atoms, const double *pos_host, const int32_t *species_host,
                      const double *box_host, int rebuild, double *energy_host, float *forces_host,
                      double *virial_host);

/*
 * n_steps of velocity-Verlet NVE with time step dt_fs.  List rebuilds:
 *   rebuild_every > 0   every `rebuild_every` steps of the context's running step counter
 *   rebuild_every = 0   never
 *   rebuild_every < 0   displacement-triggered, the policy of the paper's MD runs (Section 4.2: the criterion is
 *                       checked every five steps and the list rebuilt only when required): every -rebuild_every
 *                       steps the host reads a device flag (one stream synchronisation) and rebuilds if some atom
 *                       has moved more than 0.8 * skin/2 since the last build.  The hard limit skin/2 still raises
 *                       MLIP_ERR_SKIN_EXCEEDED in mlip_sync_status().
 * Needs a prior mlip_build_neighbors; evaluates forces first if none are current.
 * Does not synchronise unless rebuild_every < 0; device-side problems surface in mlip_sync_status().
 */
int mlip_step(mlip_ctx *ctx, int n_steps, double dt_fs, int rebuild_every, void *stream);

/*
 * n_steps of NVT dynamics at t_target_K: a Nose-Hoover chain of three thermostats (damping time t_damp_fs, N_f = 3N - 3,
 * Martyna-Tuckerman-Tobias-Klein integration: thermostat half step, velocity-Verlet step, thermostat half step) around
 * the same force evaluation.  Section 4.2 runs its MD in the NVT ensemble at 300 K without naming the thermostat; the
 * chain thermostat is the reading taken.  rebuild_every as in mlip_step.  The thermostat state lives in the context
 * (zero at creation) and carries over between calls.  Per step it adds two kinetic-energy reductions, two one-thread
 * kernels and one velocity scaling to the NVE step.
 */
int mlip_step_nvt(mlip_ctx *ctx, int n_steps, double dt_fs, int rebuild_every, double t_target_K, double t_damp_fs,
                  void *stream);
/*
 * Thermostat velocities and positions (host [3] each) and the thermostat's part of the conserved quantity
 * (sum Q_k v_eta_k^2 / 2 + N_f kT eta_1 + kT (eta_2 + eta_3), eV, with the parameters of the last mlip_step_nvt).
 * Synchronises.  mlip_reset_thermostat zeroes the state.
 */
int mlip_get_thermostat(mlip_ctx *ctx, double *v_eta_host, double *eta_host, double *energy_host);
int mlip_reset_thermostat(mlip_ctx *ctx);

/* Number of list builds since mlip_create (initial builds, in-step rebuilds, host-entry rebuilds). */
int mlip_get_rebuilds(const mlip_ctx *ctx, int64_t *n_builds_host);

/* Positions / velocities in the caller's order (dev [N][3] double, may be NULL); step counter (host). */
int mlip_get_state(mlip_ctx *ctx, double *pos, double *vel, int64_t *step_host, void *stream);
/*
 * The inverse of mlip_get_state + mlip_get_thermostat, for checkpoint / resume: positions (as mlip_set_positions: the
 * lists are kept), velocities (dev [N][3] double, caller's order; either may be NULL = unchanged), the running step
 * counter (it decides when fixed-interval rebuilds fall), and the thermostat state (host [3] each, NULL = unchanged).
 * To resume on a fresh context: mlip_create, mlip_build_neighbors with the saved positions, then mlip_set_state with
 * pos = NULL.  With force_mode = 1 the continued trajectory is bit-identical to the uninterrupted one provided the
 * state was saved right after a step on which the lists were rebuilt (the resumed context builds its lists from the
 * saved positions; between rebuilds the original run's lists were built from earlier positions, hold the pairs in
 * another order, and the fp32 per-atom sums then round differently).
 */
int mlip_set_state(mlip_ctx *ctx, const double *pos, const double *vel, int64_t step, const double *v_eta_host,
                   const double *eta_host, void *stream);
/* Potential energy of the last evaluation and kinetic energy now (dev [1] each, may be NULL). */
int mlip_get_energies(mlip_ctx *ctx, double *e_pot, double *e_kin, void *stream);

/* Synchronise the stream of the last call, return the first device-side error (or MLIP_OK), clear it. */
int mlip_sync_status(mlip_ctx *ctx);

/* Counters for reports: list entries, pairs inside r_cut at the last evaluation (syncs), kernels launched. */
int mlip_get_counters(mlip_ctx *ctx, int64_t *n_list_entries, int64_t *n_pairs_in_cutoff, int64_t *n_launches);
/*
 * CUDA-event time of the fused-kernel launches since the last reset: number of launches timed
 * and their summed duration in ms (each launch is bracketed by its own event pair on the
 * launching stream; the most recent 256 launches are kept).  Synchronises on the last event.
 */
int mlip_kernel_time(mlip_ctx *ctx, int64_t *n_launches, double *total_ms, int reset);

/*
 * Device time (CUDA events on the launching streams, ms) of the three parts of the path since the last reset:
 * list builds (binning + count + fill), fused-kernel launches, integrator kernels (kicks, drift, thermostat).
 * Each part keeps its last 256 records.  Waits for the recorded events; reset != 0 clears all three (and the
 * record of mlip_kernel_time).  Any pointer may be NULL.
 */
int mlip_get_timings(mlip_ctx *ctx, double *ms_build_host, double *ms_kernel_host, double *ms_integrate_host, int reset);

/*
 * Diagnostic: rebuild the lists at the current positions the way an in-step rebuild does (single traversal, no
 * synchronisation, capacity as it stands) with the look-back wait of the offset scan limited to `spin_limit` polls and,
 * if unpublished_tile >= 0, with that 64-atom tile withholding its look-back word.  Its successor's wait then runs out:
 * the kernel must still finish, raise MLIP_ERR_NEIGHBOR_OVERFLOW in the status word and leave every list range inside
 * the array.  The lists are unusable afterwards until the next mlip_build_neighbors.  For tests of the failure path only.
 */
int mlip_debug_rebuild(mlip_ctx *ctx, int spin_limit, int64_t unpublished_tile, void *stream);

/*
 * Measured fp32 fused-multiply-add rate of `device` in TFLOP/s (FMA = 2): a kernel of independent FMA chains on every SM,
 * best of four timed launches (CUDA events, default stream; about 10 ms in all).  The fused kernel is bound by the fp32
 * pipes (Section 3.4 discusses compute throughput, not bandwidth, as its limit), so reports quote its achieved rate
 * against this number taken in the same process, next to the nominal lanes x clock figure.  Synchronises.
 */
int mlip_measure_fp32_peak(int device, double *tflops_host);

size_t mlip_resident_bytes(const mlip_ctx *ctx);   /* device bytes the context holds */
const char *mlip_last_error(const mlip_ctx *ctx);  /* text of the last failure (ctx may be NULL) */
void mlip_destroy(mlip_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* MLIP_H */
