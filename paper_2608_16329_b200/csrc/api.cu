// C ABI (include/mlip.h): context life cycle, buffer management and the host-side
// sequencing of the kernels.  No torch types, no exceptions across the boundary.
#include <math.h>
#include <new>
#include <string.h>
#include <vector>

#include "common.cuh"
#include "scan.cuh"

using namespace mlip;

static thread_local std::string g_last_error;

static int fail(mlip_ctx *c, int code, const char *msg) {
    if (c) c->err = msg;
    g_last_error = msg;
    return code;
}

template <typename T>
static int dev_alloc(mlip_ctx *c, T **p, size_t count) {
    *p = nullptr;
    cudaError_t e = cudaMalloc((void **)p, sizeof(T) * (count ? count : 1));
    if (e != cudaSuccess) {
        cudaGetLastError();
        c->err = std::string("cudaMalloc: ") + cudaGetErrorString(e);
        return MLIP_ERR_OOM;
    }
    c->resident += sizeof(T) * (count ? count : 1);
    return MLIP_OK;
}

template <typename T>
static void dev_free(mlip_ctx *c, T **p, size_t count) {
    if (*p) {
        cudaFree(*p);
        c->resident -= sizeof(T) * (count ? count : 1);
        *p = nullptr;
    }
}

static void free_atoms(mlip_ctx *c) {
    const size_t n = (size_t)c->cap_atoms;
    dev_free(c, &c->pos4, n); dev_free(c, &c->pos4_src, n);
    dev_free(c, &c->vel, 3 * n); dev_free(c, &c->vel_src, 3 * n);
    dev_free(c, &c->user_of, n); dev_free(c, &c->user_src, n);
    dev_free(c, &c->force, n); dev_free(c, &c->disp, 3 * n); dev_free(c, &c->e_atom, n);
    dev_free(c, &c->center_order, n); dev_free(c, &c->cell_of, n);
    dev_free(c, &c->nbr_count, n); dev_free(c, &c->nbr_near, n); dev_free(c, &c->nbr_off, n + 1);
    if (c->cfg.precision == 1) { dev_free(c, &c->force_d, 3 * n); dev_free(c, &c->e_atom_d, n); }
    if (c->cfg.force_mode == 1) dev_free(c, &c->force_fx, 3 * n);
    dev_free(c, &c->tile_state, n / 64 + 2);
    if (c->cfg.list_format == 1) dev_free(c, &c->cell_id, n);
    c->cap_atoms = 0;
}

static void free_cells(mlip_ctx *c) {
    const size_t nc = (size_t)c->cap_cells, C = (size_t)c->cfg.n_species;
    dev_free(c, &c->cell_count, nc + 1); dev_free(c, &c->cell_start, nc + 1); dev_free(c, &c->cell_fill, nc + 1);
    dev_free(c, &c->bin_count, C * nc + 1); dev_free(c, &c->bin_start, C * nc + 1);
    c->cap_cells = 0;
}

static int ensure_capacity(mlip_ctx *c, int64_t n, int64_t n_cells) {
    int rc;
    if (n > c->cap_atoms) {
        free_atoms(c);
        const size_t m = (size_t)n;
#define TRY_ALLOC(p, cnt) if ((rc = dev_alloc(c, &(p), (cnt))) != MLIP_OK) return rc
        TRY_ALLOC(c->pos4, m); TRY_ALLOC(c->pos4_src, m);
        TRY_ALLOC(c->vel, 3 * m); TRY_ALLOC(c->vel_src, 3 * m);
        TRY_ALLOC(c->user_of, m); TRY_ALLOC(c->user_src, m);
        TRY_ALLOC(c->force, m); TRY_ALLOC(c->disp, 3 * m); TRY_ALLOC(c->e_atom, m);
        TRY_ALLOC(c->center_order, m); TRY_ALLOC(c->cell_of, m);
        TRY_ALLOC(c->nbr_count, m); TRY_ALLOC(c->nbr_near, m); TRY_ALLOC(c->nbr_off, m + 1);
        if (c->cfg.precision == 1) { TRY_ALLOC(c->force_d, 3 * m); TRY_ALLOC(c->e_atom_d, m); }
        if (c->cfg.force_mode == 1) TRY_ALLOC(c->force_fx, 3 * m);
        TRY_ALLOC(c->tile_state, m / 64 + 2);
        if (c->cfg.list_format == 1) TRY_ALLOC(c->cell_id, m);
        c->cap_atoms = n;
    }
    if (n_cells > c->cap_cells) {
        free_cells(c);
        const size_t nc = (size_t)n_cells, C = (size_t)c->cfg.n_species;
        TRY_ALLOC(c->cell_count, nc + 1); TRY_ALLOC(c->cell_start, nc + 1); TRY_ALLOC(c->cell_fill, nc + 1);
        TRY_ALLOC(c->bin_count, C * nc + 1); TRY_ALLOC(c->bin_start, C * nc + 1);
        c->cap_cells = n_cells;
    }
    int64_t need = scan_tmp_items(n > (int64_t)c->cfg.n_species * n_cells ? n : (int64_t)c->cfg.n_species * n_cells);
    if (need > c->scan_tmp_cap) {
        dev_free(c, &c->scan_tmp, (size_t)c->scan_tmp_cap);
        TRY_ALLOC(c->scan_tmp, (size_t)need);
        c->scan_tmp_cap = need;
    }
#undef TRY_ALLOC
    return MLIP_OK;
}

// Row-major cell vectors -> edge lengths; only orthorhombic cells aligned with the axes are compiled in.
static int box_edges(mlip_ctx *c, const double *cell, double *edges) {
    for (int a = 0; a < 3; ++a)
        for (int b = 0; b < 3; ++b)
            if (a != b && cell[3 * a + b] != 0.0) return fail(c, MLIP_ERR_UNSUPPORTED, "triclinic cells are not supported: off-diagonal cell-vector components must be zero");
    for (int a = 0; a < 3; ++a) edges[a] = cell[3 * a + a];
    return MLIP_OK;
}

static int set_grid(mlip_ctx *c, const double *box) {
    const double rl = c->cfg.r_cut + c->cfg.skin;
    CellGrid g;
    int64_t n_cells = 1;
    for (int a = 0; a < 3; ++a) {
        if (!(box[a] >= 2.0 * rl) || !isfinite(box[a])) return fail(c, MLIP_ERR_BOX_TOO_SMALL, "box edge shorter than 2 (r_cut + skin)");
        g.n[a] = (int)floor(box[a] / rl);
        if (g.n[a] < 1) g.n[a] = 1;
        g.box[a] = box[a];
        g.half[a] = 0.5 * box[a];
        g.inv_edge[a] = g.n[a] / box[a];
        n_cells *= g.n[a];
    }
    if (n_cells > 2000000000LL) return fail(c, MLIP_ERR_UNSUPPORTED, "too many cells");
    g.n_cells = (int)n_cells;
    c->grid = g;
    return MLIP_OK;
}

extern "C" {

int mlip_create(mlip_ctx **out, const mlip_config *cfg, const double *enc_w, size_t n_enc, const double *head_w,
                size_t n_head, const double *mass) {
    if (!out) return fail(nullptr, MLIP_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (!cfg || !enc_w || !head_w || !mass) return fail(nullptr, MLIP_ERR_INVALID_ARG, "NULL argument");
    if (cfg->n_species < 1 || cfg->n_species > MAX_SPECIES) return fail(nullptr, MLIP_ERR_UNSUPPORTED, "n_species must be 1..8");
    if (cfg->basis < 0 || cfg->basis > 1) return fail(nullptr, MLIP_ERR_INVALID_ARG, "basis must be 0 (irreducible) or 1 (canonical)");
    if (cfg->precision == 1) {
        if (!f64_shape_supported(cfg->k, cfg->l_max, cfg->basis))
            return fail(nullptr, MLIP_ERR_UNSUPPORTED, "the fp64 path is compiled for the irreducible basis with k in {16, 32, 64} x l_max in {1, 2, 3} and "
                                                       "k = 32 x l_max in {4, 5}, and for the canonical basis with k in {32, 64} x l_max in {1, 2, 3}");
    } else if (cfg->k < 1 || cfg->k > K_RADIAL || cfg->l_max < 0 || cfg->l_max > 3 || cfg->basis != 0) {
        return fail(nullptr, MLIP_ERR_UNSUPPORTED, "the fp32 path is compiled for k = 32, l_max = 3, irreducible basis (smaller k and l_max run in that "
                                                   "shape with the missing channels and orders zero); other shapes: precision = 1");
    }
    if (cfg->head_hidden != HEAD_H || cfg->head_layers != HEAD_L) return fail(nullptr, MLIP_ERR_UNSUPPORTED, "only a 4 x 64 head is compiled in");
    if (cfg->enc_hidden < 1 || cfg->enc_layers < 1) return fail(nullptr, MLIP_ERR_INVALID_ARG, "bad encoder shape");
    if (!(cfg->r_cut > 0.0) || !(cfg->skin >= 0.0)) return fail(nullptr, MLIP_ERR_INVALID_ARG, "bad r_cut or skin");
    if (cfg->enc_conditioning < 0 || cfg->enc_conditioning > 2 || cfg->head_conditioning < 0 || cfg->head_conditioning > 1)
        return fail(nullptr, MLIP_ERR_INVALID_ARG, "bad enc_conditioning or head_conditioning");
    if (cfg->force_mode < 0 || cfg->force_mode > 1) return fail(nullptr, MLIP_ERR_INVALID_ARG, "force_mode must be 0 (atomics) or 1 (deterministic)");
    if (cfg->force_mode == 1 && cfg->precision == 1) return fail(nullptr, MLIP_ERR_UNSUPPORTED, "the deterministic force mode is compiled for the fp32 path only");
    if (cfg->envelope < 0 || cfg->envelope > 1) return fail(nullptr, MLIP_ERR_INVALID_ARG, "envelope must be 0 (cosine) or 1 (quintic)");
    if (cfg->list_format < 0 || cfg->list_format > 1) return fail(nullptr, MLIP_ERR_INVALID_ARG, "list_format must be 0 (int32 indices) or 1 (16-bit cell-relative codes)");
    // Species conditioning (Section 3.2.2): the kernels always index C*C encoder tables and C heads; the variants
    // with fewer networks are expanded here by repeating the shared ones.
    const int C = cfg->n_species;
    const size_t enc_net = (size_t)2 * cfg->enc_hidden + (size_t)(cfg->enc_layers - 1) * ((size_t)cfg->enc_hidden * cfg->enc_hidden + cfg->enc_hidden) +
                           (size_t)cfg->k * cfg->enc_hidden + cfg->k;
    const size_t n_enc_nets = cfg->enc_conditioning == 0 ? (size_t)C * C : cfg->enc_conditioning == 1 ? (size_t)C : 1;
    const size_t n_head_nets = cfg->head_conditioning == 0 ? (size_t)C : 1;
    if (n_enc != n_enc_nets * enc_net) return fail(nullptr, MLIP_ERR_INVALID_ARG, "encoder weight count does not match shape and conditioning");
    const size_t head_net = head_net_size((cfg->l_max + 1) * cfg->k);
    if (n_head != n_head_nets * head_net) return fail(nullptr, MLIP_ERR_INVALID_ARG, "head weight count does not match shape and conditioning");
    std::vector<double> enc_full, head_full;
    try {
        if (cfg->enc_conditioning != 0) enc_full.resize((size_t)C * C * enc_net);
        if (cfg->head_conditioning != 0) head_full.resize((size_t)C * head_net);
    } catch (const std::bad_alloc &) {
        return fail(nullptr, MLIP_ERR_OOM, "host allocation failed");
    }
    if (cfg->enc_conditioning != 0) {
        for (int si = 0; si < C; ++si)
            for (int sj = 0; sj < C; ++sj)
                memcpy(&enc_full[((size_t)si * C + sj) * enc_net], enc_w + (cfg->enc_conditioning == 1 ? (size_t)sj : 0) * enc_net, sizeof(double) * enc_net);
        enc_w = enc_full.data();
        n_enc = enc_full.size();
    }
    if (cfg->head_conditioning != 0) {
        for (int si = 0; si < C; ++si) memcpy(&head_full[(size_t)si * head_net], head_w, sizeof(double) * head_net);
        head_w = head_full.data();
    }
    for (int s = 0; s < cfg->n_species; ++s)
        if (!(mass[s] > 0.0)) return fail(nullptr, MLIP_ERR_INVALID_ARG, "mass must be positive");
    if (cfg->precision != 0 && cfg->precision != 1) return fail(nullptr, MLIP_ERR_INVALID_ARG, "precision must be 0 (fp32) or 1 (fp64)");
    // fp32 path, descriptor smaller than the compiled shape (k < 32 or l_max < 3): the fused kernel runs its own shape with
    // the extra radial channels identically zero (zero output rows of every encoder) and the extra invariants unused
    // (zero columns in the regression networks' first layer).  Same function, no saving in time: the throughput side of
    // the k and l_max ablations is measured on the fp64 kernel, which is compiled per shape.
    std::vector<double> enc_pad, head_pad;
    mlip_config padded = *cfg;
    if (cfg->precision == 0 && (cfg->k < K_RADIAL || cfg->l_max < 3)) {
        const int k = cfg->k, H = cfg->enc_hidden;
        const size_t trunk = enc_net - ((size_t)k * H + k), enc_net32 = trunk + (size_t)K_RADIAL * H + K_RADIAL;
        const size_t head_tail = head_net - (size_t)HEAD_H * (cfg->l_max + 1) * k, head_net128 = head_tail + (size_t)HEAD_H * N_INV;
        try {
            enc_pad.assign((size_t)C * C * enc_net32, 0.0);
            head_pad.assign((size_t)C * head_net128, 0.0);
        } catch (const std::bad_alloc &) {
            return fail(nullptr, MLIP_ERR_OOM, "host allocation failed");
        }
        for (int n = 0; n < C * C; ++n) {
            const double *src = enc_w + (size_t)n * enc_net;
            double *dst = &enc_pad[(size_t)n * enc_net32];
            memcpy(dst, src, sizeof(double) * trunk);
            memcpy(dst + trunk, src + trunk, sizeof(double) * (size_t)k * H);                               // W_out rows 0 .. k-1
            memcpy(dst + trunk + (size_t)K_RADIAL * H, src + trunk + (size_t)k * H, sizeof(double) * k);    // b_out
        }
        for (int n = 0; n < C; ++n) {
            const double *src = head_w + (size_t)n * head_net;
            double *dst = &head_pad[(size_t)n * head_net128];
            for (int o = 0; o < HEAD_H; ++o)
                for (int l = 0; l <= cfg->l_max; ++l)
                    memcpy(dst + (size_t)o * N_INV + (size_t)l * K_RADIAL, src + (size_t)o * (cfg->l_max + 1) * k + (size_t)l * k, sizeof(double) * k);
            memcpy(dst + (size_t)HEAD_H * N_INV, src + (size_t)HEAD_H * (cfg->l_max + 1) * k, sizeof(double) * head_tail);
        }
        enc_w = enc_pad.data(); n_enc = enc_pad.size();
        head_w = head_pad.data();
        padded.k = K_RADIAL; padded.l_max = 3;
    }

    mlip_ctx *c = new (std::nothrow) mlip_ctx();
    if (!c) return fail(nullptr, MLIP_ERR_OOM, "host allocation failed");
    c->cfg = padded;
    const bool auto_knots = c->cfg.table_knots <= 0;
    const bool f64 = c->cfg.precision == 1;
    if (auto_knots) c->cfg.table_knots = f64 ? 512 : 64;
    if (c->cfg.table_r_min <= 0.0) c->cfg.table_r_min = 1.0;
    if (c->cfg.table_tol <= 0.0) c->cfg.table_tol = f64 ? 1e-10 : 1e-6;
    if (c->cfg.table_knots > 8192 || c->cfg.table_r_min >= c->cfg.r_cut) { delete c; return fail(nullptr, MLIP_ERR_INVALID_ARG, "bad table parameters"); }

    int rc = MLIP_OK;
    cudaError_t e = cudaSetDevice(cfg->device);
    cudaDeviceProp prop;
    if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, cfg->device);
    if (e != cudaSuccess) {
        g_last_error = std::string("CUDA device unavailable: ") + cudaGetErrorString(e);
        delete c;
        return MLIP_ERR_CUDA;
    }
    c->n_sm = prop.multiProcessorCount;
    do {
        if ((rc = dev_alloc(c, &c->mass, (size_t)cfg->n_species)) != MLIP_OK) break;
        if ((rc = dev_alloc(c, &c->launch_block, (size_t)LB_COUNT)) != MLIP_OK) break;
        c->tile_counter = reinterpret_cast<int *>(c->launch_block);
        c->pair_counter = reinterpret_cast<unsigned long long *>(c->launch_block + LB_PAIR);
        c->acc_fx = reinterpret_cast<long long *>(c->launch_block + LB_ACC_FX);
        c->acc = c->launch_block + LB_ACC;
        if ((rc = dev_alloc(c, &c->status, 1)) != MLIP_OK) break;
        if ((rc = dev_alloc(c, &c->rebuild_flag, 1)) != MLIP_OK) break;
        if ((rc = dev_alloc(c, &c->far_flag, 1)) != MLIP_OK) break;
        if ((rc = dev_alloc(c, &c->nhc, 8)) != MLIP_OK) break;
        if ((rc = dev_alloc(c, &c->tile_ticket, 2)) != MLIP_OK) break;   // ticket, private overflow flag
        if ((rc = dev_alloc(c, &c->species_start, (size_t)MAX_SPECIES + 1)) != MLIP_OK) break;
        if ((rc = dev_alloc(c, &c->stage_out, 10)) != MLIP_OK) break;
        if ((rc = dev_alloc(c, &c->kin_part, 1184)) != MLIP_OK) break;
        if (cudaMallocHost((void **)&c->status_host, sizeof(int)) != cudaSuccess ||
            cudaMallocHost((void **)&c->total_host, sizeof(int64_t)) != cudaSuccess ||
            cudaMallocHost((void **)&c->rebuild_host, sizeof(int)) != cudaSuccess) {
            rc = MLIP_ERR_CUDA; c->err = "pinned host allocation failed"; break;
        }
        bool ev_ok = true;
        for (int q = 0; q < 2 * mlip_ctx::EV_POOL; ++q)
            ev_ok = ev_ok && cudaEventCreate(&c->ev[q]) == cudaSuccess && cudaEventCreate(&c->ev_build[q]) == cudaSuccess &&
                    cudaEventCreate(&c->ev_integrate[q]) == cudaSuccess;
        if (!ev_ok) { rc = MLIP_ERR_CUDA; c->err = "event creation failed"; break; }
        if (cudaMemcpy(c->mass, mass, sizeof(double) * cfg->n_species, cudaMemcpyHostToDevice) != cudaSuccess ||
            cudaMemset(c->status, 0, sizeof(int)) != cudaSuccess || cudaMemset(c->rebuild_flag, 0, sizeof(int)) != cudaSuccess ||
            cudaMemset(c->nhc, 0, sizeof(double) * 8) != cudaSuccess || cudaMemset(c->launch_block, 0, sizeof(double) * LB_COUNT) != cudaSuccess) {
            rc = MLIP_ERR_CUDA; c->err = "initial upload failed"; break;
        }
        if ((rc = f64 ? upload_head_f64(c, head_w) : upload_head(c, head_w)) != MLIP_OK) break;
        rc = build_tables(c, enc_w, n_enc);
        // automatic knot count: double until the spline meets the tolerance
        while (auto_knots && rc == MLIP_ERR_TABLE_TOLERANCE && c->cfg.table_knots < (f64 ? 8192 : 2048)) {
            c->cfg.table_knots *= 2;
            rc = build_tables(c, enc_w, n_enc);
        }
    } while (0);
    if (rc != MLIP_OK && rc != MLIP_ERR_TABLE_TOLERANCE) {
        g_last_error = c->err;
        mlip_destroy(c);
        return rc;
    }
    if (rc != MLIP_OK) g_last_error = c->err;
    *out = c;
    return rc;
}

int mlip_table_error(const mlip_ctx *c, double *err_value, double *err_deriv) {
    if (!c) return MLIP_ERR_INVALID_ARG;
    if (err_value) *err_value = c->table_err_value;
    if (err_deriv) *err_deriv = c->table_err_deriv;
    return MLIP_OK;
}

int mlip_build_neighbors(mlip_ctx *c, int64_t n, const double *pos, const int32_t *species, const double *box, void *stream) {
    return mlip_build_neighbors_ghost(c, n, 0, pos, species, box, stream);
}

int mlip_build_neighbors_ghost(mlip_ctx *c, int64_t n_owned, int64_t n_ghost, const double *pos, const int32_t *species,
                               const double *box, void *stream) {
    if (!c) return MLIP_ERR_INVALID_ARG;
    const int64_t n = n_owned + n_ghost;
    if (n_owned < 1 || n_ghost < 0 || !pos || !species || !box) return fail(c, MLIP_ERR_INVALID_ARG, "bad arguments to mlip_build_neighbors");
    if (n > (1LL << 28)) return fail(c, MLIP_ERR_UNSUPPORTED, "more than 2^28 atoms per context (the pair queue packs index and species in 32 bits)");
    cudaStream_t s = (cudaStream_t)stream;
    c->last_stream = s;
    cudaSetDevice(c->cfg.device);
    double edges[3];
    int rc = box_edges(c, box, edges);
    if (rc != MLIP_OK) return rc;
    if ((rc = set_grid(c, edges)) != MLIP_OK) return rc;
    c->built = false;
    if ((rc = ensure_capacity(c, n, c->grid.n_cells)) != MLIP_OK) return rc;
    c->n = n;
    c->n_owned = n_owned;
    if (n_ghost > 0) MLIP_CUDA_TRY(c, cudaMemsetAsync(c->e_atom, 0, sizeof(float) * n, s));   // ghosts have no E_i
    if (n_ghost > 0 && c->cfg.precision == 1) MLIP_CUDA_TRY(c, cudaMemsetAsync(c->e_atom_d, 0, sizeof(double) * n, s));
    if ((rc = launch_pack_source(c, pos, species, s)) != MLIP_OK) return rc;
    double *keep = c->vel_src;   // a NULL source makes the gather reset velocities to zero
    c->vel_src = nullptr;
    rc = launch_build(c, true, s);
    c->vel_src = keep;
    if (rc != MLIP_OK) return rc;
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->rebuild_flag, 0, sizeof(int), s));
    c->built = true;
    c->forces_current = false;
    c->n_builds += 1;
    return MLIP_OK;
}

int mlip_get_neighbors(mlip_ctx *c, int64_t *seg_ptr, int32_t *nbr, int64_t capacity, int64_t *n_entries_host, void *stream) {
    if (!c || !seg_ptr) return MLIP_ERR_INVALID_ARG;
    if (!c->built) return fail(c, MLIP_ERR_NOT_BUILT, "no neighbor lists yet");
    c->last_stream = (cudaStream_t)stream;
    cudaSetDevice(c->cfg.device);
    return launch_export(c, seg_ptr, nbr, capacity, n_entries_host, (cudaStream_t)stream);
}

int mlip_get_neighbors_noalloc(mlip_ctx *c, int64_t *seg_ptr, int32_t *nbr, int64_t capacity, int64_t *n_entries_host, void *stream) {
    if (!c || !seg_ptr) return MLIP_ERR_INVALID_ARG;
    if (!c->built) return fail(c, MLIP_ERR_NOT_BUILT, "no neighbor lists yet");
    c->last_stream = (cudaStream_t)stream;
    cudaSetDevice(c->cfg.device);
    return launch_export_noalloc(c, seg_ptr, nbr, capacity, n_entries_host, (cudaStream_t)stream);
}

int mlip_set_positions(mlip_ctx *c, const double *pos, void *stream) {
    if (!c || !pos) return MLIP_ERR_INVALID_ARG;
    if (!c->built) return fail(c, MLIP_ERR_NOT_BUILT, "no neighbor lists yet");
    c->last_stream = (cudaStream_t)stream;
    c->forces_current = false;
    return launch_set_positions(c, pos, (cudaStream_t)stream);
}

int mlip_set_velocities(mlip_ctx *c, const double *vel, void *stream) {
    if (!c || !vel) return MLIP_ERR_INVALID_ARG;
    if (!c->built) return fail(c, MLIP_ERR_NOT_BUILT, "no neighbor lists yet");
    c->last_stream = (cudaStream_t)stream;
    return launch_set_velocities(c, vel, (cudaStream_t)stream);
}

// The fused evaluation in the context's precision.
static int evaluate(mlip_ctx *c, cudaStream_t s) {
    return c->cfg.precision == 1 ? launch_megakernel_f64(c, s) : launch_megakernel(c, s);
}

int mlip_compute_f64(mlip_ctx *c, double *energy, double *forces, double *virial, double *e_atom, void *stream) {
    if (!c) return MLIP_ERR_INVALID_ARG;
    if (c->cfg.precision != 1) return fail(c, MLIP_ERR_UNSUPPORTED, "mlip_compute_f64 needs a context created with precision = 1");
    if (!c->built) return fail(c, MLIP_ERR_NOT_BUILT, "no neighbor lists yet");
    cudaStream_t s = (cudaStream_t)stream;
    c->last_stream = s;
    int rc = launch_megakernel_f64(c, s);
    if (rc != MLIP_OK) return rc;
    c->forces_current = true;
    if (energy) MLIP_CUDA_TRY(c, cudaMemcpyAsync(energy, c->acc + ACC_ENERGY, sizeof(double), cudaMemcpyDeviceToDevice, s));
    if (virial) MLIP_CUDA_TRY(c, cudaMemcpyAsync(virial, c->acc + ACC_VIRIAL, sizeof(double) * 9, cudaMemcpyDeviceToDevice, s));
    if (forces || e_atom) rc = launch_scatter_forces_f64(c, forces, e_atom, s);
    return rc;
}

int mlip_compute(mlip_ctx *c, double *energy, float *forces, double *virial, float *e_atom, void *stream) {
    if (!c) return MLIP_ERR_INVALID_ARG;
    if (!c->built) return fail(c, MLIP_ERR_NOT_BUILT, "no neighbor lists yet");
    cudaStream_t s = (cudaStream_t)stream;
    c->last_stream = s;
    int rc = evaluate(c, s);
    if (rc != MLIP_OK) return rc;
    c->forces_current = true;
    if (energy) MLIP_CUDA_TRY(c, cudaMemcpyAsync(energy, c->acc + ACC_ENERGY, sizeof(double), cudaMemcpyDeviceToDevice, s));
    if (virial) MLIP_CUDA_TRY(c, cudaMemcpyAsync(virial, c->acc + ACC_VIRIAL, sizeof(double) * 9, cudaMemcpyDeviceToDevice, s));
    if (forces || e_atom) rc = launch_scatter_forces(c, forces, e_atom, s);
    return rc;
}

int mlip_compute_host(mlip_ctx *c, int64_t n, const double *pos_host, const int32_t *species_host, const double *box_host,
                      int rebuild, double *energy_host, float *forces_host, double *virial_host) {
    if (!c || !pos_host || n < 1) return MLIP_ERR_INVALID_ARG;
    cudaStream_t s = c->last_stream;
    cudaSetDevice(c->cfg.device);
    const bool need_build = rebuild || !c->built || n != c->n;
    if (need_build && (!species_host || !box_host)) return fail(c, MLIP_ERR_INVALID_ARG, "species and box are needed to build the lists");
    int rc;
    if (n > c->stage_cap) {
        dev_free(c, &c->stage_pos, 3 * (size_t)c->stage_cap);
        dev_free(c, &c->stage_species, (size_t)c->stage_cap);
        dev_free(c, &c->stage_force, 3 * (size_t)c->stage_cap);
        c->stage_cap = 0;
        if ((rc = dev_alloc(c, &c->stage_pos, 3 * (size_t)n)) != MLIP_OK) return rc;
        if ((rc = dev_alloc(c, &c->stage_species, (size_t)n)) != MLIP_OK) return rc;
        if ((rc = dev_alloc(c, &c->stage_force, 3 * (size_t)n)) != MLIP_OK) return rc;
        c->stage_cap = n;
    }
    MLIP_CUDA_TRY(c, cudaMemcpyAsync(c->stage_pos, pos_host, sizeof(double) * 3 * n, cudaMemcpyHostToDevice, s));
    if (need_build) {
        MLIP_CUDA_TRY(c, cudaMemcpyAsync(c->stage_species, species_host, sizeof(int32_t) * n, cudaMemcpyHostToDevice, s));
        if ((rc = mlip_build_neighbors(c, n, c->stage_pos, c->stage_species, box_host, s)) != MLIP_OK) return rc;
    } else if ((rc = mlip_set_positions(c, c->stage_pos, s)) != MLIP_OK) return rc;
    if ((rc = mlip_compute(c, c->stage_out, forces_host ? c->stage_force : nullptr, c->stage_out + 1, nullptr, s)) != MLIP_OK) return rc;
    if (forces_host) MLIP_CUDA_TRY(c, cudaMemcpyAsync(forces_host, c->stage_force, sizeof(float) * 3 * n, cudaMemcpyDeviceToHost, s));
    double out[10];
    MLIP_CUDA_TRY(c, cudaMemcpyAsync(out, c->stage_out, sizeof out, cudaMemcpyDeviceToHost, s));
    MLIP_CUDA_TRY(c, cudaStreamSynchronize(s));
    if (energy_host) *energy_host = out[0];
    if (virial_host) memcpy(virial_host, out + 1, sizeof(double) * 9);
    return MLIP_OK;
}

// After a drift: rebuild the lists if the policy asks for it (fixed interval, or displacement-triggered).
static int rebuild_if_due(mlip_ctx *c, int rebuild_every, cudaStream_t s) {
    bool rebuild = rebuild_every > 0 && c->step % rebuild_every == 0;
    if (rebuild_every < 0 && c->step % -rebuild_every == 0) {   // displacement-triggered: ask the device
        MLIP_CUDA_TRY(c, cudaMemcpyAsync(c->rebuild_host, c->rebuild_flag, sizeof(int), cudaMemcpyDeviceToHost, s));
        MLIP_CUDA_TRY(c, cudaStreamSynchronize(s));
        rebuild = *c->rebuild_host != 0;
    }
    if (!rebuild) return MLIP_OK;
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->rebuild_flag, 0, sizeof(int), s));
    c->n_builds += 1;
    std::swap(c->pos4, c->pos4_src);
    std::swap(c->vel, c->vel_src);
    std::swap(c->user_of, c->user_src);
    return launch_build(c, false, s);
}

int mlip_step(mlip_ctx *c, int n_steps, double dt, int rebuild_every, void *stream) {
    if (!c || n_steps < 0 || !(dt > 0.0)) return MLIP_ERR_INVALID_ARG;
    if (!c->built) return fail(c, MLIP_ERR_NOT_BUILT, "no neighbor lists yet");
    if (c->n_owned != c->n) return fail(c, MLIP_ERR_UNSUPPORTED, "a context with ghost atoms evaluates only: the owner of the ghosts integrates them");
    cudaStream_t s = (cudaStream_t)stream;
    c->last_stream = s;
    int rc;
    if (!c->forces_current) {
        if ((rc = evaluate(c, s)) != MLIP_OK) return rc;
        c->forces_current = true;
    }
    for (int it = 0; it < n_steps; ++it) {
        if ((rc = launch_kick_drift(c, dt, s)) != MLIP_OK) return rc;
        c->step += 1;
        if ((rc = rebuild_if_due(c, rebuild_every, s)) != MLIP_OK) return rc;
        if ((rc = evaluate(c, s)) != MLIP_OK) return rc;
        if ((rc = launch_kick(c, dt, s)) != MLIP_OK) return rc;
    }
    return MLIP_OK;
}

int mlip_step_nvt(mlip_ctx *c, int n_steps, double dt, int rebuild_every, double t_target, double t_damp, void *stream) {
    if (!c || n_steps < 0 || !(dt > 0.0) || !(t_target > 0.0) || !(t_damp > 0.0)) return MLIP_ERR_INVALID_ARG;
    if (!c->built) return fail(c, MLIP_ERR_NOT_BUILT, "no neighbor lists yet");
    if (c->n < 2) return fail(c, MLIP_ERR_INVALID_ARG, "the thermostat needs at least two atoms");
    if (c->n_owned != c->n) return fail(c, MLIP_ERR_UNSUPPORTED, "a context with ghost atoms evaluates only: the owner of the ghosts integrates them");
    cudaStream_t s = (cudaStream_t)stream;
    c->last_stream = s;
    const double kB = 8.617333262e-5;   // eV/K
    c->nhc_nf = 3.0 * (double)c->n - 3.0;
    c->nhc_kT = kB * t_target;
    c->nhc_qk = c->nhc_kT * t_damp * t_damp;
    c->nhc_q1 = c->nhc_nf * c->nhc_qk;
    int rc;
    if (!c->forces_current) {
        if ((rc = evaluate(c, s)) != MLIP_OK) return rc;
        c->forces_current = true;
    }
    for (int it = 0; it < n_steps; ++it) {
        // kinetic energy of the velocities as they stand (not the previous half step's rescaled value, so that a run does
        // not depend on how it is split into calls), then the thermostat half step; its velocity factor is applied
        // inside the kick-drift kernel
        if ((rc = launch_kinetic(c, s)) != MLIP_OK) return rc;
        if ((rc = launch_nhc_half(c, c->nhc_nf, c->nhc_kT, c->nhc_q1, c->nhc_qk, dt, s)) != MLIP_OK) return rc;
        if ((rc = launch_kick_drift(c, dt, s, c->nhc + 6)) != MLIP_OK) return rc;
        c->step += 1;
        if ((rc = rebuild_if_due(c, rebuild_every, s)) != MLIP_OK) return rc;
        if ((rc = evaluate(c, s)) != MLIP_OK) return rc;
        if ((rc = launch_kick(c, dt, s)) != MLIP_OK) return rc;
        if ((rc = launch_kinetic(c, s)) != MLIP_OK) return rc;
        if ((rc = launch_nhc_half(c, c->nhc_nf, c->nhc_kT, c->nhc_q1, c->nhc_qk, dt, s)) != MLIP_OK) return rc;
        if ((rc = launch_scale_velocities(c, s)) != MLIP_OK) return rc;
    }
    return MLIP_OK;
}

int mlip_get_thermostat(mlip_ctx *c, double *v_eta_host, double *eta_host, double *energy_host) {
    if (!c) return MLIP_ERR_INVALID_ARG;
    double st[8];
    MLIP_CUDA_TRY(c, cudaStreamSynchronize(c->last_stream));
    MLIP_CUDA_TRY(c, cudaMemcpy(st, c->nhc, sizeof st, cudaMemcpyDeviceToHost));
    if (v_eta_host) memcpy(v_eta_host, st, sizeof(double) * 3);
    if (eta_host) memcpy(eta_host, st + 3, sizeof(double) * 3);
    if (energy_host)
        *energy_host = 0.5 * (c->nhc_q1 * st[0] * st[0] + c->nhc_qk * (st[1] * st[1] + st[2] * st[2])) +
                       c->nhc_nf * c->nhc_kT * st[3] + c->nhc_kT * (st[4] + st[5]);
    return MLIP_OK;
}

int mlip_reset_thermostat(mlip_ctx *c) {
    if (!c) return MLIP_ERR_INVALID_ARG;
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->nhc, 0, sizeof(double) * 8, c->last_stream));
    return MLIP_OK;
}

int mlip_get_state(mlip_ctx *c, double *pos, double *vel, int64_t *step_host, void *stream) {
    if (!c) return MLIP_ERR_INVALID_ARG;
    if (!c->built) return fail(c, MLIP_ERR_NOT_BUILT, "no atoms yet");
    c->last_stream = (cudaStream_t)stream;
    if (step_host) *step_host = c->step;
    if (pos || vel) return launch_get_state(c, pos, vel, (cudaStream_t)stream);
    return MLIP_OK;
}

int mlip_set_state(mlip_ctx *c, const double *pos, const double *vel, int64_t step, const double *v_eta_host,
                   const double *eta_host, void *stream) {
    if (!c || step < 0) return MLIP_ERR_INVALID_ARG;
    if (!c->built) return fail(c, MLIP_ERR_NOT_BUILT, "no atoms yet: build the lists from the saved positions first");
    cudaStream_t s = (cudaStream_t)stream;
    c->last_stream = s;
    int rc;
    if (pos) {
        c->forces_current = false;
        if ((rc = launch_set_positions(c, pos, s)) != MLIP_OK) return rc;
    }
    if (vel && (rc = launch_set_velocities(c, vel, s)) != MLIP_OK) return rc;
    c->step = step;
    if (v_eta_host || eta_host) {   // thermostat state {v_eta[3], eta[3]}
        double st[6];
        MLIP_CUDA_TRY(c, cudaStreamSynchronize(s));
        MLIP_CUDA_TRY(c, cudaMemcpy(st, c->nhc, sizeof st, cudaMemcpyDeviceToHost));
        if (v_eta_host) memcpy(st, v_eta_host, sizeof(double) * 3);
        if (eta_host) memcpy(st + 3, eta_host, sizeof(double) * 3);
        MLIP_CUDA_TRY(c, cudaMemcpy(c->nhc, st, sizeof st, cudaMemcpyHostToDevice));
    }
    return MLIP_OK;
}

int mlip_debug_rebuild(mlip_ctx *c, int spin_limit, int64_t unpublished_tile, void *stream) {
    if (!c || spin_limit < 1) return MLIP_ERR_INVALID_ARG;
    if (!c->built) return fail(c, MLIP_ERR_NOT_BUILT, "no neighbor lists yet");
    cudaStream_t s = (cudaStream_t)stream;
    c->last_stream = s;
    c->lookback_spin_limit = spin_limit;
    c->lookback_unpublished_tile = unpublished_tile;
    std::swap(c->pos4, c->pos4_src);
    std::swap(c->vel, c->vel_src);
    std::swap(c->user_of, c->user_src);
    int rc = launch_build(c, false, s);
    c->lookback_spin_limit = 0;
    c->lookback_unpublished_tile = -1;
    c->n_builds += 1;
    c->forces_current = false;
    return rc;
}

int mlip_get_rebuilds(const mlip_ctx *c, int64_t *n_builds_host) {
    if (!c || !n_builds_host) return MLIP_ERR_INVALID_ARG;
    *n_builds_host = c->n_builds;
    return MLIP_OK;
}

int mlip_get_energies(mlip_ctx *c, double *e_pot, double *e_kin, void *stream) {
    if (!c) return MLIP_ERR_INVALID_ARG;
    if (!c->built) return fail(c, MLIP_ERR_NOT_BUILT, "no atoms yet");
    cudaStream_t s = (cudaStream_t)stream;
    c->last_stream = s;
    if (e_pot) MLIP_CUDA_TRY(c, cudaMemcpyAsync(e_pot, c->acc + ACC_ENERGY, sizeof(double), cudaMemcpyDeviceToDevice, s));
    if (e_kin) {
        int rc = launch_kinetic(c, s);
        if (rc != MLIP_OK) return rc;
        MLIP_CUDA_TRY(c, cudaMemcpyAsync(e_kin, c->acc + ACC_KINETIC, sizeof(double), cudaMemcpyDeviceToDevice, s));
    }
    return MLIP_OK;
}

int mlip_sync_status(mlip_ctx *c) {
    if (!c) return MLIP_ERR_INVALID_ARG;
    cudaStream_t s = c->last_stream;
    MLIP_CUDA_TRY(c, cudaMemcpyAsync(c->status_host, c->status, sizeof(int), cudaMemcpyDeviceToHost, s));
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->status, 0, sizeof(int), s));
    MLIP_CUDA_TRY(c, cudaStreamSynchronize(s));
    const int f = *c->status_host;
    if (f & FLAG_NONFINITE) return fail(c, MLIP_ERR_NONFINITE, "non-finite or out-of-box position, or species out of range");
    if (f & FLAG_NEIGHBOR_OVERFLOW) return fail(c, MLIP_ERR_NEIGHBOR_OVERFLOW, "neighbor list capacity exceeded during a rebuild");
    if (f & FLAG_SKIN_EXCEEDED) return fail(c, MLIP_ERR_SKIN_EXCEEDED, "an atom moved more than skin/2 since the last list build");
    if (f & FLAG_BOUNDS) return fail(c, MLIP_ERR_CUDA, "range-checked build: an index left its array");
    if (f & FLAG_TABLE_RANGE) return fail(c, MLIP_ERR_TABLE_RANGE, "a pair came closer than table_r_min");
    return MLIP_OK;
}

int mlip_get_counters(mlip_ctx *c, int64_t *n_list_entries, int64_t *n_pairs, int64_t *n_launches) {
    if (!c) return MLIP_ERR_INVALID_ARG;
    MLIP_CUDA_TRY(c, cudaStreamSynchronize(c->last_stream));
    if (n_list_entries) {
        *n_list_entries = 0;
        if (c->built) MLIP_CUDA_TRY(c, cudaMemcpy(n_list_entries, c->nbr_off + c->n, sizeof(int64_t), cudaMemcpyDeviceToHost));
    }
    if (n_pairs) {
        unsigned long long v = 0;
        MLIP_CUDA_TRY(c, cudaMemcpy(&v, c->pair_counter, sizeof v, cudaMemcpyDeviceToHost));
        *n_pairs = (int64_t)v;
    }
    if (n_launches) *n_launches = c->launches;
    return MLIP_OK;
}

int mlip_kernel_time(mlip_ctx *c, int64_t *n_launches, double *total_ms, int reset) {
    if (!c) return MLIP_ERR_INVALID_ARG;
    const int64_t kept = c->ev_count < mlip_ctx::EV_POOL ? c->ev_count : mlip_ctx::EV_POOL;
    double total = 0.0;
    for (int64_t q = 0; q < kept; ++q) {
        const int slot = (int)((c->ev_count - 1 - q) % mlip_ctx::EV_POOL);
        float ms = 0.f;
        MLIP_CUDA_TRY(c, cudaEventSynchronize(c->ev[2 * slot + 1]));
        MLIP_CUDA_TRY(c, cudaEventElapsedTime(&ms, c->ev[2 * slot], c->ev[2 * slot + 1]));
        total += ms;
    }
    if (n_launches) *n_launches = kept;
    if (total_ms) *total_ms = total;
    if (reset) c->ev_count = 0;
    return MLIP_OK;
}

// Sum of the last min(count, EV_POOL) event pairs of a pool, in ms.
static int pool_total(mlip_ctx *c, cudaEvent_t *pool, int64_t count, double *total_ms) {
    const int64_t kept = count < mlip_ctx::EV_POOL ? count : mlip_ctx::EV_POOL;
    double total = 0.0;
    for (int64_t q = 0; q < kept; ++q) {
        const int slot = (int)((count - 1 - q) % mlip_ctx::EV_POOL);
        float ms = 0.f;
        MLIP_CUDA_TRY(c, cudaEventSynchronize(pool[2 * slot + 1]));
        MLIP_CUDA_TRY(c, cudaEventElapsedTime(&ms, pool[2 * slot], pool[2 * slot + 1]));
        total += ms;
    }
    *total_ms = total;
    return MLIP_OK;
}

int mlip_get_timings(mlip_ctx *c, double *ms_build, double *ms_kernel, double *ms_integrate, int reset) {
    if (!c) return MLIP_ERR_INVALID_ARG;
    double b = 0.0, k = 0.0, i = 0.0;
    int rc;
    if ((rc = pool_total(c, c->ev_build, c->build_count, &b)) != MLIP_OK) return rc;
    if ((rc = pool_total(c, c->ev, c->ev_count, &k)) != MLIP_OK) return rc;
    if ((rc = pool_total(c, c->ev_integrate, c->integrate_count, &i)) != MLIP_OK) return rc;
    if (ms_build) *ms_build = b;
    if (ms_kernel) *ms_kernel = k;
    if (ms_integrate) *ms_integrate = i;
    if (reset) { c->build_count = 0; c->ev_count = 0; c->integrate_count = 0; }
    return MLIP_OK;
}

#ifdef MLIP_PHASE_CLOCKS
int mlip_debug_acc(mlip_ctx *c, double *out16) {   // profiling builds only
    cudaDeviceSynchronize();
    return cudaMemcpy(out16, c->acc, sizeof(double) * ACC_COUNT, cudaMemcpyDeviceToHost) == cudaSuccess ? MLIP_OK : MLIP_ERR_CUDA;
}
#endif

size_t mlip_resident_bytes(const mlip_ctx *c) { return c ? c->resident : 0; }

const char *mlip_last_error(const mlip_ctx *c) { return c ? c->err.c_str() : g_last_error.c_str(); }

void mlip_destroy(mlip_ctx *c) {
    if (!c) return;
    cudaSetDevice(c->cfg.device);
    cudaDeviceSynchronize();
    free_atoms(c);
    free_cells(c);
    cudaFree(c->nbr); cudaFree(c->scan_tmp); cudaFree(c->head_w); cudaFree(c->table); cudaFree(c->mass);
    cudaFree(c->head_w_d); cudaFree(c->table_d);
    cudaFree(c->launch_block); cudaFree(c->status); cudaFree(c->rebuild_flag); cudaFree(c->far_flag); cudaFree(c->nhc); cudaFree(c->tile_ticket);
    cudaFree(c->species_start); cudaFree(c->stage_pos); cudaFree(c->stage_species); cudaFree(c->stage_force);
    cudaFree(c->stage_out); cudaFree(c->kin_part);
    if (c->status_host) cudaFreeHost(c->status_host);
    if (c->total_host) cudaFreeHost(c->total_host);
    if (c->rebuild_host) cudaFreeHost(c->rebuild_host);
    for (int q = 0; q < 2 * mlip_ctx::EV_POOL; ++q) {
        if (c->ev[q]) cudaEventDestroy(c->ev[q]);
        if (c->ev_build[q]) cudaEventDestroy(c->ev_build[q]);
        if (c->ev_integrate[q]) cudaEventDestroy(c->ev_integrate[q]);
    }
    delete c;
}

}  // extern "C"
