// Cell binning and neighbor-list construction (Section 3.1.1: N(i) = atoms within a
// cutoff of atom i; the paper delegates this to the MD code's binning algorithm,
// Section 4.1.4).  Everything runs on the device:
//   cell id per atom -> counting sort into cell order (ties broken by species, then by the
//   caller's index, so the internal order is reproducible) -> per-species processing order
//   -> two passes (count, fill) of a warp-per-atom scan over the 27 surrounding cells.
// The inclusion test is fp64 with separately rounded operations, so the set of pairs is
// identical to a plain CPU evaluation of the same expression.
#include "common.cuh"
#include "scan.cuh"

namespace mlip {

__device__ __forceinline__ int cell_coord(double x, double inv_edge, int n) {
    int c = (int)floor(x * inv_edge);
    return c < 0 ? 0 : (c >= n ? n - 1 : c);
}

// ---- compact list format ----
// With atoms stored in cell order a neighbor j of atom i lies in one of the 27 cells around i's cell, so an entry can
// be coded in 16 bits: the cell's number in the traversal order (0..26: x, y, z offsets ascending) in the top 5 bits, j's
// position inside that cell in the low 11 (a cell holds at most MAX_CELL_ATOMS = 1,024 atoms).  Decoding needs the build-time
// cell of i (cell_id) and the cell starts.  Half the bytes of the int32 list, the bulk of the resident footprint.
// Used when mlip_config.list_format = 1 and every dimension has at least three cells.
// One list entry in the format of the output array: the index itself, or its 16-bit code.
template <typename OUT>
__device__ __forceinline__ OUT list_entry(int j, int it, int cell_beg) {
    if (sizeof(OUT) == 2) return (OUT)((it << L16_SHIFT) | (j - cell_beg));
    return (OUT)j;
}

__global__ void k_pack_source(const double *__restrict__ pos, const int32_t *__restrict__ species, int64_t n,
                              int n_species, double4 *__restrict__ pos4, int32_t *__restrict__ user, int *status) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    int s = species[i];
    if (s < 0 || s >= n_species) { atomicOr(status, FLAG_NONFINITE); s = 0; }
    pos4[i] = make_double4(pos[3 * i], pos[3 * i + 1], pos[3 * i + 2], (double)s);
    user[i] = (int32_t)i;
}

__global__ void k_cell_id(const double4 *__restrict__ pos4, int64_t n, CellGrid g, int32_t *__restrict__ cell_of,
                          int32_t *__restrict__ cell_count, int *status) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    double4 p = pos4[i];
    bool ok = (p.x >= 0.0 && p.x < g.box[0]) && (p.y >= 0.0 && p.y < g.box[1]) && (p.z >= 0.0 && p.z < g.box[2]);
    if (!ok) atomicOr(status, FLAG_NONFINITE);
    int cx = ok ? cell_coord(p.x, g.inv_edge[0], g.n[0]) : 0;
    int cy = ok ? cell_coord(p.y, g.inv_edge[1], g.n[1]) : 0;
    int cz = ok ? cell_coord(p.z, g.inv_edge[2], g.n[2]) : 0;
    int c = (cx * g.n[1] + cy) * g.n[2] + cz;
    cell_of[i] = c;
    atomicAdd(&cell_count[c], 1);
}

__global__ void k_place(const int32_t *__restrict__ cell_of, int64_t n, const int32_t *__restrict__ cell_start,
                        int32_t *__restrict__ cell_fill, int32_t *__restrict__ slot_src) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    int c = cell_of[i];
    slot_src[cell_start[c] + atomicAdd(&cell_fill[c], 1)] = (int32_t)i;
}

// One thread per cell: order the cell's atoms by (species, caller index) and count them per species.
// A cell holding more than MAX_CELL_ATOMS atoms (a collapsed or diverged configuration: thousands of atoms in a cube of
// one list radius) is not sorted -- the insertion sort is quadratic in one thread -- and raises FLAG_NONFINITE, which
// makes the list kernels and the fused kernels that follow return at once.
constexpr int MAX_CELL_ATOMS = 1024;
__global__ void k_sort_cells(int n_cells, int n_species, const int32_t *__restrict__ cell_start,
                             int32_t *__restrict__ slot_src, const double4 *__restrict__ pos4_src,
                             const int32_t *__restrict__ user_src, int32_t *__restrict__ bin_count, int *status, int32_t n_owned) {
    // (bin_count counts the atoms that will be central atoms: caller indices below n_owned; the others are ghosts)
    int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= n_cells) return;
    int beg = cell_start[c], end = cell_start[c + 1];
    int cnt[MAX_SPECIES] = {0};
    if (end - beg > MAX_CELL_ATOMS) {
        atomicOr(status, FLAG_NONFINITE);
        for (int a = beg; a < end; ++a) { const int src = slot_src[a]; cnt[(int)pos4_src[src].w] += user_src[src] < n_owned; }
        for (int s = 0; s < n_species; ++s) bin_count[(int64_t)s * n_cells + c] = cnt[s];
        return;
    }
    for (int a = beg; a < end; ++a) {
        int src = slot_src[a];
        int sa = (int)pos4_src[src].w;
        long long key = ((long long)sa << 32) | (unsigned)user_src[src];
        cnt[sa] += user_src[src] < n_owned;
        int b = a - 1;
        while (b >= beg) {
            int sb_src = slot_src[b];
            long long kb = ((long long)(int)pos4_src[sb_src].w << 32) | (unsigned)user_src[sb_src];
            if (kb <= key) break;
            slot_src[b + 1] = sb_src;
            --b;
        }
        slot_src[b + 1] = src;
    }
    for (int s = 0; s < n_species; ++s) bin_count[(int64_t)s * n_cells + c] = cnt[s];
}

__global__ void k_gather(int64_t n, const int32_t *__restrict__ slot_src, const double4 *__restrict__ pos4_src,
                         const double *__restrict__ vel_src, const int32_t *__restrict__ user_src,
                         double4 *__restrict__ pos4, double *__restrict__ vel, int32_t *__restrict__ user_of,
                         float *__restrict__ disp, const int32_t *__restrict__ cell_of, int32_t *__restrict__ cell_id, CellGrid g) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    int src = slot_src[i];
    if (cell_id) cell_id[i] = pack_cell(g, cell_of[src]);   // build-time cell of the atom in the internal order (compact lists)
    pos4[i] = pos4_src[src];
    user_of[i] = user_src[src];
    for (int a = 0; a < 3; ++a) {
        vel[3 * i + a] = vel_src ? vel_src[3 * (int64_t)src + a] : 0.0;
        disp[3 * i + a] = 0.f;
    }
}

// One thread per cell: the cell's atoms (already species-ordered) go to their (species, cell) bins.
__global__ void k_center_order(int n_cells, int n_species, const int32_t *__restrict__ cell_start,
                               const double4 *__restrict__ pos4, const int32_t *__restrict__ bin_start,
                               int32_t *__restrict__ center_order, int32_t *__restrict__ species_start,
                               const int32_t *__restrict__ user_of, int32_t n_owned) {
    int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c <= n_species) species_start[c] = c < n_species ? bin_start[(int64_t)c * n_cells] : bin_start[(int64_t)n_species * n_cells];
    if (c >= n_cells) return;
    int beg = cell_start[c], end = cell_start[c + 1];
    int prev = -1, r = 0;
    for (int a = beg; a < end; ++a) {
        int s = (int)pos4[a].w;
        if (s != prev) { prev = s; r = 0; }
        if (user_of[a] < n_owned) center_order[bin_start[(int64_t)s * n_cells + c] + r++] = a;   // ghosts are never central atoms
    }
}

// Warp per atom over the surrounding cells.  FILL = false counts, FILL = true writes the list.
// Lanes 0..26 fetch the atom ranges of the (up to) 27 cells in one round trip; the cells are then visited
// in a fixed order (x, y, z offsets ascending: the order of the list) with the positions of the next
// cell requested before the current one is tested, so that an atom costs a few load latencies instead of 54.
template <bool FILL>
__global__ void __launch_bounds__(256) k_neighbors(int64_t n, CellGrid g, double rl2, const double4 *__restrict__ pos4,
                                                   const int32_t *__restrict__ cell_start, int32_t *__restrict__ nbr_count,
                                                   const int64_t *__restrict__ nbr_off, int32_t *__restrict__ nbr,
                                                   int64_t nbr_cap, int *status, float near2, int32_t *__restrict__ nbr_near,
                                                   const int32_t *__restrict__ user_of, int32_t n_owned) {
    const int lane = threadIdx.x & 31;
    int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (i >= n || (*status & FLAG_NONFINITE)) return;   // a broken configuration is not traversed (see k_sort_cells)
    if (user_of[i] >= n_owned) {   // a ghost is listed by others but has no list of its own
        if (!FILL && lane == 0) { nbr_count[i] = 0; nbr_near[i] = 0; }
        return;
    }
    const double4 pi = pos4[i];
    // this lane's cell: offsets (ox, oy, oz) = (lane / 9, lane / 3 % 3, lane % 3); dimensions with fewer than
    // three cells list each cell once
    int cb = 0, ce = 0;
    {
        const int o[3] = {lane / 9, (lane / 3) % 3, lane % 3};
        const double p[3] = {pi.x, pi.y, pi.z};
        int cc[3];
        bool ok = lane < 27;
#pragma unroll
        for (int a = 0; a < 3; ++a) {
            const int na = g.n[a];
            const int c0 = cell_coord(p[a], g.inv_edge[a], na);
            int c = c0 + o[a] - 1;
            c = c < 0 ? c + na : (c >= na ? c - na : c);
            if (na < 3) { c = o[a]; ok = ok && o[a] < na; }
            cc[a] = c;
        }
        if (ok) {
            const int c = (cc[0] * g.n[1] + cc[1]) * g.n[2] + cc[2];
            cb = cell_start[c]; ce = cell_start[c + 1];
        }
    }
    const float boxf[3] = {(float)g.box[0], (float)g.box[1], (float)g.box[2]};
    const float halff[3] = {(float)g.half[0], (float)g.half[1], (float)g.half[2]};
    const float rl2_lo = (float)(rl2 * (1.0 - 1e-5)), rl2_hi = (float)(rl2 * (1.0 + 1e-5));
    int64_t off = 0;
    bool writable = true;
    int total = 0;
    if (FILL) {
        off = nbr_off[i];
        total = (int)(nbr_off[i + 1] - off);
        writable = nbr_off[i + 1] <= nbr_cap;
        if (!writable && lane == 0) atomicOr(status, FLAG_NEIGHBOR_OVERFLOW);
    }
    int cnt = 0, cn = 0;   // hits so far, near hits so far (near hits fill the list from the front, far hits from the back)
    int beg = __shfl_sync(0xffffffffu, cb, 0), end = __shfl_sync(0xffffffffu, ce, 0);
    double4 pj_next = make_double4(0.0, 0.0, 0.0, 0.0);
    if (beg + lane < end) pj_next = pos4[beg + lane];
    for (int it = 0; it < 27; ++it) {
        const int cur_beg = beg, cur_end = end;
        double4 pj = pj_next;
        if (it + 1 < 27) {   // request the first chunk of the next cell
            beg = __shfl_sync(0xffffffffu, cb, it + 1);
            end = __shfl_sync(0xffffffffu, ce, it + 1);
            if (beg + lane < end) pj_next = pos4[beg + lane];
        }
        for (int base = cur_beg; base < cur_end; base += 32) {
            const int j = base + lane;
            if (base != cur_beg && j < cur_end) pj = pos4[j];
            bool hit = false;
            float d2f = 0.f;
            if (j < cur_end && j != i) {
                const double ex = __dsub_rn(pj.x, pi.x), ey = __dsub_rn(pj.y, pi.y), ez = __dsub_rn(pj.z, pi.z);
                // fp32 screen: the squared distance to ~1e-6 relative decides every candidate that is not within
                // 1e-5 of the list radius; only those few take the exact, individually rounded fp64 predicate
                float fx = fabsf((float)ex), fy = fabsf((float)ey), fz = fabsf((float)ez);
                fx = fx > halff[0] ? boxf[0] - fx : fx;
                fy = fy > halff[1] ? boxf[1] - fy : fy;
                fz = fz > halff[2] ? boxf[2] - fz : fz;
                d2f = fx * fx + fy * fy + fz * fz;
                if (d2f < rl2_lo) hit = true;
                else if (d2f <= rl2_hi) {
                    const double dx = min_image(ex, g.box[0], g.half[0]);
                    const double dy = min_image(ey, g.box[1], g.half[1]);
                    const double dz = min_image(ez, g.box[2], g.half[2]);
                    const double d2 = __dadd_rn(__dadd_rn(__dmul_rn(dx, dx), __dmul_rn(dy, dy)), __dmul_rn(dz, dz));
                    hit = d2 < rl2;
                }
            }
            const bool near = hit && d2f < near2;
            const unsigned m = __ballot_sync(0xffffffffu, hit), mn = __ballot_sync(0xffffffffu, near), below = (1u << lane) - 1u;
            if (FILL && hit && writable)
                nbr[off + (near ? cn + __popc(mn & below) : total - 1 - (cnt - cn + __popc(m & ~mn & below)))] = j;
            cnt += __popc(m);
            cn += __popc(mn);
        }
    }
    if (!FILL && lane == 0) { nbr_count[i] = cnt; nbr_near[i] = cn; }
}

// Positions relative to the lower corner of the atom's own cell, in fp32 (|x_rel| < cell edge, so the rounding is ~5e-7
// Angstrom whatever the box size).  Lives in the force array, which is idle during a build.
__global__ void k_rel_pos(int64_t n, CellGrid g, const double4 *__restrict__ pos4, float4 *__restrict__ rel) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const double4 p = pos4[i];
    const double x[3] = {p.x, p.y, p.z};
    float r[3];
#pragma unroll
    for (int a = 0; a < 3; ++a) {
        const int c = cell_coord(x[a], g.inv_edge[a], g.n[a]);
        r[a] = (float)(x[a] - (double)c * (g.box[a] / g.n[a]));
    }
    rel[i] = make_float4(r[0], r[1], r[2], 0.f);
}

// The same traversal for grids with at least three cells per dimension, on the cell-relative fp32 positions: the
// separation is x_rel(j) - x_rel(i) + (cell offset) * edge -- the cell offset already names the periodic image, so no
// minimum-image step and no fp64 arithmetic per candidate.  Candidates within 1e-5 of the list radius (the fp32 distance is
// good to ~1e-6) are decided by the exact fp64 predicate on the full positions, so the lists are the same bit for bit.
template <bool FILL, typename OUT>
__global__ void __launch_bounds__(256) k_neighbors_rel(int64_t n, CellGrid g, double rl2, const double4 *__restrict__ pos4,
                                                       const float4 *__restrict__ rel, const int32_t *__restrict__ cell_start,
                                                       int32_t *__restrict__ nbr_count, const int64_t *__restrict__ nbr_off,
                                                       OUT *__restrict__ nbr, int64_t nbr_cap, int *status, float near2,
                                                       int32_t *__restrict__ nbr_near, const int32_t *__restrict__ user_of, int32_t n_owned) {
    const int lane = threadIdx.x & 31;
    int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (i >= n || (*status & FLAG_NONFINITE)) return;
    if (user_of[i] >= n_owned) {
        if (!FILL && lane == 0) { nbr_count[i] = 0; nbr_near[i] = 0; }
        return;
    }
    const double4 pi = pos4[i];
    const float4 ri = rel[i];
    int cb = 0, ce = 0;
    if (lane < 27) {
        const int o[3] = {lane / 9, (lane / 3) % 3, lane % 3};
        const double p[3] = {pi.x, pi.y, pi.z};
        int cc[3];
#pragma unroll
        for (int a = 0; a < 3; ++a) {
            const int na = g.n[a];
            int c = cell_coord(p[a], g.inv_edge[a], na) + o[a] - 1;
            cc[a] = c < 0 ? c + na : (c >= na ? c - na : c);
        }
        const int c = (cc[0] * g.n[1] + cc[1]) * g.n[2] + cc[2];
        cb = cell_start[c]; ce = cell_start[c + 1];
    }
    const float edge[3] = {(float)(g.box[0] / g.n[0]), (float)(g.box[1] / g.n[1]), (float)(g.box[2] / g.n[2])};
    const float rl2_lo = (float)(rl2 * (1.0 - 1e-5)), rl2_hi = (float)(rl2 * (1.0 + 1e-5));
    int64_t off = 0;
    bool writable = true;
    int total = 0;
    if (FILL) {
        off = nbr_off[i];
        total = (int)(nbr_off[i + 1] - off);
        writable = nbr_off[i + 1] <= nbr_cap;
        if (!writable && lane == 0) atomicOr(status, FLAG_NEIGHBOR_OVERFLOW);
    }
    int cnt = 0, cn = 0;
    int beg = __shfl_sync(0xffffffffu, cb, 0), end = __shfl_sync(0xffffffffu, ce, 0);
    float4 rj_next = make_float4(0.f, 0.f, 0.f, 0.f);
    if (beg + lane < end) rj_next = rel[beg + lane];
#pragma unroll
    for (int it = 0; it < 27; ++it) {
        const int cur_beg = beg, cur_end = end;
        float4 rj = rj_next;
        if (it + 1 < 27) {   // request the first chunk of the next cell
            beg = __shfl_sync(0xffffffffu, cb, it + 1);
            end = __shfl_sync(0xffffffffu, ce, it + 1);
            if (beg + lane < end) rj_next = rel[beg + lane];
        }
        // separation = x_rel(j) + shift, shift = (cell offset) * edge - x_rel(i)
        const float sx = (float)(it / 9 - 1) * edge[0] - ri.x;
        const float sy = (float)((it / 3) % 3 - 1) * edge[1] - ri.y;
        const float sz = (float)(it % 3 - 1) * edge[2] - ri.z;
        for (int base = cur_beg; base < cur_end; base += 32) {
            const int j = base + lane;
            if (base != cur_beg && j < cur_end) rj = rel[j];
            bool hit = false;
            float d2f = 0.f;
            if (j < cur_end && j != i) {
                const float dx = rj.x + sx, dy = rj.y + sy, dz = rj.z + sz;
                d2f = dx * dx + dy * dy + dz * dz;
                if (d2f < rl2_lo) hit = true;
                else if (d2f <= rl2_hi) {
                    const double4 pj = pos4[j];
                    const double ex = min_image(__dsub_rn(pj.x, pi.x), g.box[0], g.half[0]);
                    const double ey = min_image(__dsub_rn(pj.y, pi.y), g.box[1], g.half[1]);
                    const double ez = min_image(__dsub_rn(pj.z, pi.z), g.box[2], g.half[2]);
                    const double d2 = __dadd_rn(__dadd_rn(__dmul_rn(ex, ex), __dmul_rn(ey, ey)), __dmul_rn(ez, ez));
                    hit = d2 < rl2;
                }
            }
            const bool near = hit && d2f < near2;
            const unsigned m = __ballot_sync(0xffffffffu, hit), mn = __ballot_sync(0xffffffffu, near), below = (1u << lane) - 1u;
            if (FILL && hit && writable)
                nbr[off + (near ? cn + __popc(mn & below) : total - 1 - (cnt - cn + __popc(m & ~mn & below)))] = list_entry<OUT>(j, it, cur_beg);
            cnt += __popc(m);
            cn += __popc(mn);
        }
    }
    if (!FILL && lane == 0) { nbr_count[i] = cnt; nbr_near[i] = cn; }
}

// ---- one-pass variant for in-step rebuilds ----
// Count and fill in a single traversal: a CTA takes a tile of 64 consecutive atoms (8 per warp), collects each atom's hits
// in shared memory while it counts, obtains the tile's list offset from a decoupled look-back scan over the tiles before
// it (tile aggregate / inclusive prefix published in one 64-bit word, tiles handed out by a ticket so that every
// predecessor belongs to a CTA that is already running), and then copies the lists out in full rows.  Offsets are the same exclusive prefix sums the two-pass build produces, so the lists are identical.
// Every wait is bounded: after `spin_limit` polls (OP_SPIN in production) the tile raises FLAG_NEIGHBOR_OVERFLOW, publishes
// what it has and goes on.  Offsets are clamped to the capacity and a list that crosses it is cut short, so whatever the
// outcome every [nbr_off[i], nbr_off[i+1]) lies inside the array and holds atom indices.
constexpr int OP_PER_WARP = 8;
constexpr int OP_TILE = 8 * OP_PER_WARP;
static_assert(OP_TILE == 64, "the in-tile scan handles two counts per lane of one warp");
constexpr int OP_SPIN = 1 << 18;

__device__ __forceinline__ bool rel_hit(const float4 &rj, float sx, float sy, float sz, float rl2_lo, float rl2_hi, double rl2,
                                        const double4 &pi, const double4 *__restrict__ pos4, int j, const CellGrid &g, float &d2f) {
    const float dx = rj.x + sx, dy = rj.y + sy, dz = rj.z + sz;
    d2f = dx * dx + dy * dy + dz * dz;
    if (d2f < rl2_lo) return true;
    if (d2f > rl2_hi) return false;
    const double4 pj = pos4[j];
    const double ex = min_image(__dsub_rn(pj.x, pi.x), g.box[0], g.half[0]);
    const double ey = min_image(__dsub_rn(pj.y, pi.y), g.box[1], g.half[1]);
    const double ez = min_image(__dsub_rn(pj.z, pi.z), g.box[2], g.half[2]);
    return __dadd_rn(__dadd_rn(__dmul_rn(ex, ex), __dmul_rn(ey, ey)), __dmul_rn(ez, ez)) < rl2;
}

// atom ranges of the 27 cells around position p, one cell per lane (lanes 27.. get an empty range)
__device__ __forceinline__ void cell_ranges(const double4 &p4, const CellGrid &g, const int32_t *__restrict__ cell_start, int lane,
                                            int &cb, int &ce) {
    cb = 0; ce = 0;
    if (lane < 27) {
        const int o[3] = {lane / 9, (lane / 3) % 3, lane % 3};
        const double p[3] = {p4.x, p4.y, p4.z};
        int cc[3];
#pragma unroll
        for (int a = 0; a < 3; ++a) {
            const int na = g.n[a];
            int c = cell_coord(p[a], g.inv_edge[a], na) + o[a] - 1;
            cc[a] = c < 0 ? c + na : (c >= na ? c - na : c);
        }
        const int c = (cc[0] * g.n[1] + cc[1]) * g.n[2] + cc[2];
        cb = cell_start[c]; ce = cell_start[c + 1];
    }
}

// One atom's traversal for the one-pass build.  Near hits (inside near2) go to out[0], out[1], ..., far hits to out[top],
// out[top - 1], ...; only positions below `limit` are written.  Shared-memory pass: top = capacity - 1 (if the list is
// longer than the buffer the two ends collide and the list is traversed again); global pass: top = list length - 1.
// Returns the number of hits, and the number of near hits in `n_near`.
template <typename OUT, typename ENTRY>
__device__ __forceinline__ int onepass_traverse(int64_t i, const CellGrid &g, double rl2, const float (&edge)[3], float rl2_lo, float rl2_hi,
                                                const double4 *__restrict__ pos4, const float4 *__restrict__ rel,
                                                const int32_t *__restrict__ cell_start, int lane, OUT *out, int top, int limit,
                                                float near2, int &n_near) {
    // OUT = type of the buffer written here (int32 in shared memory), ENTRY = format of the list (int32 or uint16)
    const double4 pi = pos4[i];
    const float4 ri = rel[i];
    int cb, ce;
    cell_ranges(pi, g, cell_start, lane, cb, ce);
    int cnt = 0, cn = 0;
    int beg = __shfl_sync(0xffffffffu, cb, 0), end = __shfl_sync(0xffffffffu, ce, 0);
    float4 rj_next = make_float4(0.f, 0.f, 0.f, 0.f);
    if (beg + lane < end) rj_next = rel[beg + lane];
#pragma unroll
    for (int it = 0; it < 27; ++it) {
        const int cur_beg = beg, cur_end = end;
        float4 rj = rj_next;
        if (it + 1 < 27) {
            beg = __shfl_sync(0xffffffffu, cb, it + 1);
            end = __shfl_sync(0xffffffffu, ce, it + 1);
            if (beg + lane < end) rj_next = rel[beg + lane];
        }
        const float sx = (float)(it / 9 - 1) * edge[0] - ri.x;
        const float sy = (float)((it / 3) % 3 - 1) * edge[1] - ri.y;
        const float sz = (float)(it % 3 - 1) * edge[2] - ri.z;
        for (int base = cur_beg; base < cur_end; base += 32) {
            const int j = base + lane;
            if (base != cur_beg && j < cur_end) rj = rel[j];
            float d2f = 0.f;
            const bool hit = j < cur_end && j != i && rel_hit(rj, sx, sy, sz, rl2_lo, rl2_hi, rl2, pi, pos4, j, g, d2f);
            const bool near = hit && d2f < near2;
            const unsigned m = __ballot_sync(0xffffffffu, hit), mn = __ballot_sync(0xffffffffu, near), below = (1u << lane) - 1u;
            const int slot = near ? cn + __popc(mn & below) : top - (cnt - cn + __popc(m & ~mn & below));
            if (hit && slot >= 0 && slot < limit) out[slot] = (OUT)list_entry<ENTRY>(j, it, cur_beg);
            cnt += __popc(m);
            cn += __popc(mn);
        }
    }
    n_near = cn;
    return cnt;
}

constexpr int OP_BUF = 160;   // hits kept per atom in shared memory; a longer list is traversed again straight into global memory

template <typename ENTRY>
__global__ void __launch_bounds__(256) k_neighbors_onepass(int64_t n, CellGrid g, double rl2, const double4 *__restrict__ pos4,
                                                           const float4 *__restrict__ rel, const int32_t *__restrict__ cell_start,
                                                           int64_t *__restrict__ nbr_off, ENTRY *__restrict__ nbr, int64_t nbr_cap,
                                                           int *status, unsigned long long *tile_state, int *ticket,
                                                           const int *global_status, int spin_limit, long long unpublished_tile,
                                                           float near2, int32_t *__restrict__ nbr_near,
                                                           const int32_t *__restrict__ user_of, int32_t n_owned) {
    // `unpublished_tile` >= 0 (diagnostic builds of the lists only) names a tile that never publishes its look-back word,
    // so that its successor's bounded wait can be seen to run out; -1 in production.
    if (*global_status & FLAG_NONFINITE) return;   // a broken configuration is not traversed (see k_sort_cells)
    // look-back word: flag in the top two bits (0 empty, 1 tile aggregate, 2 inclusive prefix), value below
    constexpr unsigned long long OP_AGG = 1ull << 62, OP_INC = 2ull << 62, OP_VAL = (1ull << 62) - 1;
    extern __shared__ int32_t s_hits[];   // [OP_TILE][OP_BUF]
    __shared__ int s_cnt[OP_TILE], s_near[OP_TILE];
    __shared__ long long s_off[OP_TILE];
    __shared__ long long s_prefix, s_total;
    __shared__ int s_tile;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_tile = atomicAdd(ticket, 1);
    __syncthreads();
    const int64_t tile = s_tile, first = tile * OP_TILE;
    const float edge[3] = {(float)(g.box[0] / g.n[0]), (float)(g.box[1] / g.n[1]), (float)(g.box[2] / g.n[2])};
    const float rl2_lo = (float)(rl2 * (1.0 - 1e-5)), rl2_hi = (float)(rl2 * (1.0 + 1e-5));

    // ---- traversal: count, keep the hits ----
    for (int a = 0; a < OP_PER_WARP; ++a) {
        const int slot = warp * OP_PER_WARP + a;
        const int64_t i = first + slot;
        int cnt = 0, cn = 0;
        if (i < n && user_of[i] < n_owned)   // (a ghost has no list of its own)
            cnt = onepass_traverse<int32_t, ENTRY>(i, g, rl2, edge, rl2_lo, rl2_hi, pos4, rel, cell_start, lane, s_hits + slot * OP_BUF, OP_BUF - 1, OP_BUF, near2, cn);
        if (lane == 0) { s_cnt[slot] = cnt; s_near[slot] = cn; }
    }
    __syncthreads();

    // ---- offsets: scan inside the tile, look back over the tiles before it ----
    if (warp == 0) {
        const int c0 = s_cnt[2 * lane], c1 = s_cnt[2 * lane + 1];
        long long incl = c0 + c1;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const long long v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        s_off[2 * lane] = incl - c0 - c1;
        s_off[2 * lane + 1] = incl - c1;
        const long long aggregate = __shfl_sync(0xffffffffu, incl, 31);
        volatile unsigned long long *state = tile_state;
        long long prefix = 0;
        if (tile > 0) {
            if (lane == 0 && tile != unpublished_tile) state[tile] = OP_AGG | (unsigned long long)aggregate;
            int64_t hi = tile - 1;
            int spins = 0;
            for (;;) {   // windows of 32 predecessors, nearest first
                const int64_t p = hi - lane;
                unsigned long long v = OP_INC;
                if (p >= 0) v = state[p];
                const unsigned flag = (unsigned)(v >> 62);
                const unsigned inc = __ballot_sync(0xffffffffu, flag == 2), empty = __ballot_sync(0xffffffffu, flag == 0);
                const int first_inc = inc ? __ffs(inc) - 1 : 32;
                const unsigned need = first_inc >= 31 ? 0xffffffffu : ((2u << first_inc) - 1u);
                if (empty & need) {   // a tile in the window has not published yet
                    if (++spins > spin_limit) { if (lane == 0) atomicOr(status, FLAG_NEIGHBOR_OVERFLOW); break; }
                    __nanosleep(200);
                    continue;
                }
                long long val = (lane <= first_inc && p >= 0) ? (long long)(v & OP_VAL) : 0;
#pragma unroll
                for (int o = 16; o; o >>= 1) val += __shfl_xor_sync(0xffffffffu, val, o);
                prefix += val;
                if (first_inc < 32) break;
                hi -= 32;
            }
        }
        if (lane == 0) {
            if (tile != unpublished_tile) state[tile] = OP_INC | (unsigned long long)(prefix + aggregate);
            s_prefix = prefix;
            s_total = prefix + aggregate;
        }
    }
    __syncthreads();
    const long long tile_off = s_prefix;
    if (first + OP_TILE >= n && threadIdx.x == 0) nbr_off[n] = s_total < nbr_cap ? s_total : nbr_cap;   // the last tile closes the offsets

    // ---- write the lists: full rows from shared memory ----
    for (int a = 0; a < OP_PER_WARP; ++a) {
        const int slot = warp * OP_PER_WARP + a;
        const int64_t i = first + slot;
        if (i >= n) break;
        const long long off = tile_off + s_off[slot];
        const int cnt = s_cnt[slot];
        int fit = cnt;   // entries of this list that the array still holds
        if (off + cnt > nbr_cap) {
            if (lane == 0) atomicOr(status, FLAG_NEIGHBOR_OVERFLOW);
            fit = off < nbr_cap ? (int)(nbr_cap - off) : 0;
        }
        const int near = s_near[slot];
        if (lane == 0) { nbr_off[i] = off < nbr_cap ? off : nbr_cap; nbr_near[i] = near < fit ? near : fit; }
        if (fit == 0) continue;
        if (cnt <= OP_BUF) {   // near hits sit at the front of the buffer, far hits at its back
            const int32_t *src = s_hits + slot * OP_BUF;
            for (int e = lane; e < fit; e += 32) nbr[off + e] = (ENTRY)src[e < near ? e : e + (OP_BUF - cnt)];
        } else {
            int cn;
            onepass_traverse<ENTRY, ENTRY>(i, g, rl2, edge, rl2_lo, rl2_hi, pos4, rel, cell_start, lane, nbr + off, cnt - 1, fit, near2, cn);
        }
    }
}

// ---- canonical export: caller's indices, species-segmented, ascending ----
// Entry e of atom i's list as an internal index, whatever the list format (cell_id = nullptr: plain indices).
struct ListView {
    const int32_t *nbr;
    const uint16_t *nbr16;
    const int32_t *cell_id, *cell_start;
    CellGrid grid;
    __device__ __forceinline__ int at(int64_t i, int64_t e) const {
        if (!nbr16) return nbr[e];
        const int code = nbr16[e];
        return cell_start[neighbor_cell(grid, cell_id[i], code >> L16_SHIFT)] + (code & L16_MASK);
    }
};

__global__ void k_export_count(int64_t n, int n_species, const int64_t *__restrict__ nbr_off, ListView lv,
                               const double4 *__restrict__ pos4, const int32_t *__restrict__ user_of,
                               int32_t *__restrict__ seg_count) {
    const int lane = threadIdx.x & 31;
    int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (i >= n) return;
    int cnt[MAX_SPECIES] = {0};
    for (int64_t e = nbr_off[i] + lane; e < nbr_off[i + 1]; e += 32) cnt[(int)pos4[lv.at(i, e)].w]++;
    int64_t row = (int64_t)user_of[i] * n_species;
    for (int s = 0; s < n_species; ++s) {
        int v = cnt[s];
        for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) seg_count[row + s] = v;
    }
}

__global__ void k_export_fill(int64_t n, int n_species, const int64_t *__restrict__ nbr_off, ListView lv,
                              const double4 *__restrict__ pos4, const int32_t *__restrict__ user_of,
                              const int64_t *__restrict__ seg_ptr, int32_t *__restrict__ out) {
    const int lane = threadIdx.x & 31;
    int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (i >= n) return;
    const int64_t beg = nbr_off[i], end = nbr_off[i + 1];
    const int64_t row = (int64_t)user_of[i] * n_species;
    for (int64_t e = beg + lane; e < end; e += 32) {
        int j = lv.at(i, e);
        int sj = (int)pos4[j].w, uj = user_of[j];
        int rank = 0;   // entries of the same species with a smaller caller index
        for (int64_t f = beg; f < end; ++f) {
            int jf = lv.at(i, f);
            rank += ((int)pos4[jf].w == sj) && (user_of[jf] < uj);
        }
        out[seg_ptr[row + sj] + rank] = uj;
    }
}

static inline unsigned blocks_for(int64_t n, int per_block) { return (unsigned)((n + per_block - 1) / per_block); }

static ListView list_view(const mlip_ctx *c) {
    ListView lv;
    lv.nbr = c->nbr;
    lv.nbr16 = c->list16 ? reinterpret_cast<const uint16_t *>(c->nbr) : nullptr;
    lv.cell_id = c->cell_id; lv.cell_start = c->cell_start; lv.grid = c->grid;
    return lv;
}

int launch_pack_source(mlip_ctx *c, const double *pos, const int32_t *species, cudaStream_t s) {
    k_pack_source<<<blocks_for(c->n, 256), 256, 0, s>>>(pos, species, c->n, c->cfg.n_species, c->pos4_src, c->user_src, c->status);
    c->launches += 1;
    MLIP_CUDA_TRY(c, cudaGetLastError());
    return MLIP_OK;
}

// A synchronising build that met a non-finite or out-of-box position, a species out of range or an over-full cell: the
// list kernels have not run, so there is nothing to size a list from.  Reports it now and clears the flag.
static int refuse_broken_input(mlip_ctx *c, cudaStream_t s) {
    timing_end(c->ev_build, c->build_count, s);
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->status, 0, sizeof(int), s));
    c->err = "non-finite or out-of-box position, species out of range, or more than 1024 atoms in one cell";
    return MLIP_ERR_NONFINITE;
}

// Sort (pos4_src, vel_src, user_src) into cell order and build the lists.
int launch_build(mlip_ctx *c, bool allow_sync_grow, cudaStream_t s) {
    timing_begin(c->ev_build, c->build_count, s);
    const int64_t n = c->n;
    const CellGrid &g = c->grid;
    const int C = c->cfg.n_species;
    const double rl = c->cfg.r_cut + c->cfg.skin;
    // entries farther than r_cut + skin / 2 at build time form the back part of each list: they cannot come inside r_cut
    // before some atom has moved skin / 4, and the fused kernels skip them until then (far_flag, raised by the integrator)
    const double rn = c->cfg.r_cut + 0.5 * c->cfg.skin;
    const float near2 = c->cfg.skin > 0.0 ? (float)(rn * rn * (1.0 + 1e-5)) : 3.0e38f;
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->far_flag, 0, sizeof(int), s));
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->cell_count, 0, sizeof(int32_t) * (g.n_cells + 1), s));
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->cell_fill, 0, sizeof(int32_t) * (g.n_cells + 1), s));
    k_cell_id<<<blocks_for(n, 256), 256, 0, s>>>(c->pos4_src, n, g, c->cell_of, c->cell_count, c->status);
    exclusive_scan<int32_t, int32_t>(c->cell_count, c->cell_start, g.n_cells, c->scan_tmp, s);
    // nbr_count doubles as the slot -> source map until the lists are counted
    int32_t *slot_src = c->nbr_count;
    k_place<<<blocks_for(n, 256), 256, 0, s>>>(c->cell_of, n, c->cell_start, c->cell_fill, slot_src);
    k_sort_cells<<<blocks_for(g.n_cells, 128), 128, 0, s>>>(g.n_cells, C, c->cell_start, slot_src, c->pos4_src, c->user_src, c->bin_count, c->status, (int32_t)c->n_owned);
    k_gather<<<blocks_for(n, 256), 256, 0, s>>>(n, slot_src, c->pos4_src, c->vel_src, c->user_src, c->pos4, c->vel, c->user_of, c->disp, c->cell_of, c->cell_id, g);
    exclusive_scan<int32_t, int32_t>(c->bin_count, c->bin_start, (int64_t)C * g.n_cells, c->scan_tmp, s);
    int nthreads_co = g.n_cells > C + 1 ? g.n_cells : C + 1;
    k_center_order<<<blocks_for(nthreads_co, 128), 128, 0, s>>>(g.n_cells, C, c->cell_start, c->pos4, c->bin_start, c->center_order, c->species_start, c->user_of, (int32_t)c->n_owned);
    // grids of at least 3 x 3 x 3 cells take the fp32 cell-relative traversal (positions staged in the idle force array)
    const bool rel = g.n[0] >= 3 && g.n[1] >= 3 && g.n[2] >= 3;
    float4 *relpos = c->force;
    // entry format of this build: 16-bit cell-relative codes if asked for and the grid has 27 distinct cells around every
    // cell, else plain indices.  A change of format gives up the old array (its capacity is counted in entries).
    const bool list16 = c->cfg.list_format == 1 && rel && std::max(g.n[0], std::max(g.n[1], g.n[2])) <= CELL_PACK_MAX;
    if (list16 != c->list16 && c->nbr) {
        cudaFree(c->nbr);
        c->resident -= (c->list16 ? sizeof(uint16_t) : sizeof(int32_t)) * c->nbr_cap;
        c->nbr = nullptr; c->nbr_cap = 0;
    }
    c->list16 = list16;
    const size_t entry_bytes = list16 ? sizeof(uint16_t) : sizeof(int32_t);
    uint16_t *nbr16 = reinterpret_cast<uint16_t *>(c->nbr);
    // Single traversal whenever a list array exists: always for in-step rebuilds (capacity as it stands, overflow -> status
    // bit), and for a synchronising build as a first try whose overflow flag is private and sends it to the two-pass path.
    bool rel_ready = false;
    if (rel && c->tile_state && c->nbr_cap > 0) {
        const int64_t n_tiles = (n + OP_TILE - 1) / OP_TILE;
        MLIP_CUDA_TRY(c, cudaMemsetAsync(c->tile_state, 0, sizeof(unsigned long long) * (n_tiles + 1), s));
        MLIP_CUDA_TRY(c, cudaMemsetAsync(c->tile_ticket, 0, 2 * sizeof(int), s));
        k_rel_pos<<<blocks_for(n, 256), 256, 0, s>>>(n, g, c->pos4, relpos);
        rel_ready = true;
        int *flag = allow_sync_grow ? c->tile_ticket + 1 : c->status;
        const int spin = c->lookback_spin_limit > 0 ? c->lookback_spin_limit : OP_SPIN;
        if (list16)
            k_neighbors_onepass<uint16_t><<<(unsigned)n_tiles, 256, sizeof(int32_t) * OP_TILE * OP_BUF, s>>>(
                n, g, rl * rl, c->pos4, relpos, c->cell_start, c->nbr_off, nbr16, c->nbr_cap, flag, c->tile_state, c->tile_ticket, c->status, spin,
                c->lookback_unpublished_tile, near2, c->nbr_near, c->user_of, (int32_t)c->n_owned);
        else
            k_neighbors_onepass<int32_t><<<(unsigned)n_tiles, 256, sizeof(int32_t) * OP_TILE * OP_BUF, s>>>(
                n, g, rl * rl, c->pos4, relpos, c->cell_start, c->nbr_off, c->nbr, c->nbr_cap, flag, c->tile_state, c->tile_ticket, c->status, spin,
                c->lookback_unpublished_tile, near2, c->nbr_near, c->user_of, (int32_t)c->n_owned);
        c->launches += 5 + 2 * 3 + 2;   // cell id, place, sort, gather, centre order; two scans; relative positions, lists
        MLIP_CUDA_TRY(c, cudaGetLastError());
        bool done = true;
        if (allow_sync_grow) {
            int overflow = 0;
            MLIP_CUDA_TRY(c, cudaMemcpyAsync(c->total_host, c->nbr_off + n, sizeof(int64_t), cudaMemcpyDeviceToHost, s));
            MLIP_CUDA_TRY(c, cudaMemcpyAsync(&overflow, c->tile_ticket + 1, sizeof(int), cudaMemcpyDeviceToHost, s));
            MLIP_CUDA_TRY(c, cudaMemcpyAsync(c->status_host, c->status, sizeof(int), cudaMemcpyDeviceToHost, s));
            MLIP_CUDA_TRY(c, cudaStreamSynchronize(s));
            if (*c->status_host & FLAG_NONFINITE) return refuse_broken_input(c, s);
            done = overflow == 0 && *c->total_host < c->nbr_cap;   // the kernel clamps the total to the capacity
            if (done) c->n_entries = *c->total_host;
        }
        if (done) {
            timing_end(c->ev_build, c->build_count, s);
            return MLIP_OK;
        }
    }
    if (rel) {
        if (!rel_ready) k_rel_pos<<<blocks_for(n, 256), 256, 0, s>>>(n, g, c->pos4, relpos);
        k_neighbors_rel<false, int32_t><<<blocks_for(n * 32, 256), 256, 0, s>>>(n, g, rl * rl, c->pos4, relpos, c->cell_start, c->nbr_count, nullptr, nullptr, 0, c->status, near2, c->nbr_near, c->user_of, (int32_t)c->n_owned);
        c->launches += 1;
    } else
        k_neighbors<false><<<blocks_for(n * 32, 256), 256, 0, s>>>(n, g, rl * rl, c->pos4, c->cell_start, c->nbr_count, nullptr, nullptr, 0, c->status, near2, c->nbr_near, c->user_of, (int32_t)c->n_owned);
    exclusive_scan<int32_t, int64_t>(c->nbr_count, c->nbr_off, n, c->scan_tmp, s);
    c->launches += 5 + 1 + 3 * 3;   // cell id, place, sort, gather, centre order; count; three scans
    MLIP_CUDA_TRY(c, cudaGetLastError());
    if (allow_sync_grow) {
        MLIP_CUDA_TRY(c, cudaMemcpyAsync(c->total_host, c->nbr_off + n, sizeof(int64_t), cudaMemcpyDeviceToHost, s));
        MLIP_CUDA_TRY(c, cudaMemcpyAsync(c->status_host, c->status, sizeof(int), cudaMemcpyDeviceToHost, s));
        MLIP_CUDA_TRY(c, cudaStreamSynchronize(s));
        if (*c->status_host & FLAG_NONFINITE) return refuse_broken_input(c, s);
        c->n_entries = *c->total_host;
        if (c->n_entries > c->nbr_cap) {
            int64_t want = c->n_entries + c->n_entries / 8 + 1024;
            if (c->nbr) { cudaFree(c->nbr); c->resident -= entry_bytes * c->nbr_cap; c->nbr = nullptr; c->nbr_cap = 0; }
            MLIP_CUDA_TRY(c, cudaMalloc(&c->nbr, entry_bytes * want));
            c->nbr_cap = want;
            c->resident += entry_bytes * want;
            nbr16 = reinterpret_cast<uint16_t *>(c->nbr);
        }
    }
    if (rel && list16)
        k_neighbors_rel<true, uint16_t><<<blocks_for(n * 32, 256), 256, 0, s>>>(n, g, rl * rl, c->pos4, relpos, c->cell_start, c->nbr_count, c->nbr_off, nbr16, c->nbr_cap, c->status, near2, c->nbr_near, c->user_of, (int32_t)c->n_owned);
    else if (rel)
        k_neighbors_rel<true, int32_t><<<blocks_for(n * 32, 256), 256, 0, s>>>(n, g, rl * rl, c->pos4, relpos, c->cell_start, c->nbr_count, c->nbr_off, c->nbr, c->nbr_cap, c->status, near2, c->nbr_near, c->user_of, (int32_t)c->n_owned);
    else
        k_neighbors<true><<<blocks_for(n * 32, 256), 256, 0, s>>>(n, g, rl * rl, c->pos4, c->cell_start, c->nbr_count, c->nbr_off, c->nbr, c->nbr_cap, c->status, near2, c->nbr_near, c->user_of, (int32_t)c->n_owned);
    c->launches += 1;
    timing_end(c->ev_build, c->build_count, s);
    MLIP_CUDA_TRY(c, cudaGetLastError());
    return MLIP_OK;
}

// The lists cannot be exported while the status word says that the last in-step rebuild did not complete them.
static int lists_whole(mlip_ctx *c, cudaStream_t s) {
    MLIP_CUDA_TRY(c, cudaMemcpyAsync(c->status_host, c->status, sizeof(int), cudaMemcpyDeviceToHost, s));
    MLIP_CUDA_TRY(c, cudaStreamSynchronize(s));
    if (*c->status_host & FLAG_NONFINITE) { c->err = "neighbor export: the configuration is broken (see mlip_sync_status)"; return MLIP_ERR_NONFINITE; }
    if (*c->status_host & FLAG_NEIGHBOR_OVERFLOW) { c->err = "neighbor export: the last rebuild overflowed the list (see mlip_sync_status)"; return MLIP_ERR_NEIGHBOR_OVERFLOW; }
    return MLIP_OK;
}

int launch_export(mlip_ctx *c, int64_t *seg_ptr, int32_t *nbr, int64_t capacity, int64_t *n_entries_host, cudaStream_t s) {
    const int64_t n = c->n;
    const int C = c->cfg.n_species;
    int whole = lists_whole(c, s);
    if (whole != MLIP_OK) return whole;
    int32_t *seg_count = nullptr;
    MLIP_CUDA_TRY(c, cudaMalloc(&seg_count, sizeof(int32_t) * (size_t)(n * C + 1)));
    int64_t *tmp = nullptr;
    if (cudaMalloc(&tmp, sizeof(int64_t) * (size_t)scan_tmp_items(n * C)) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(seg_count);
        c->err = "neighbor export: cudaMalloc of the scan scratch failed";
        return MLIP_ERR_OOM;
    }
    k_export_count<<<blocks_for(n * 32, 256), 256, 0, s>>>(n, C, c->nbr_off, list_view(c), c->pos4, c->user_of, seg_count);
    exclusive_scan<int32_t, int64_t>(seg_count, seg_ptr, n * C, tmp, s);
    int rc = MLIP_OK;
    cudaError_t e = cudaMemcpyAsync(c->total_host, seg_ptr + n * C, sizeof(int64_t), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e == cudaSuccess) {
        if (n_entries_host) *n_entries_host = *c->total_host;
        if (*c->total_host > capacity || !nbr) rc = MLIP_ERR_NEIGHBOR_OVERFLOW;
        else {
            k_export_fill<<<blocks_for(n * 32, 256), 256, 0, s>>>(n, C, c->nbr_off, list_view(c), c->pos4, c->user_of, seg_ptr, nbr);
            e = cudaStreamSynchronize(s);
        }
    }
    c->launches += 5;
    cudaFree(seg_count);
    cudaFree(tmp);
    if (e != cudaSuccess) { c->err = cudaGetErrorString(e); return MLIP_ERR_CUDA; }
    if (rc != MLIP_OK) c->err = "neighbor export: capacity too small";
    return rc;
}

}  // namespace mlip

// ---- allocation-free variant of the canonical export ----
//
// For callers that must not allocate device memory while they run: code inside a region where
// cudaMalloc would serialise or fail (a latency-critical MD loop that owns a fixed memory budget, a
// plug-in running under a host application whose allocator it may not touch), or a process whose
// device memory is already fully committed.  The two temporaries of the export (per-(atom, species)
// counts and the partial sums of the prefix scan) live in a file-scope device array instead of
// fresh cudaMalloc blocks.  Every GPU that loads the library holds the array until the process exits.
namespace mlip {

constexpr int64_t NOALLOC_MAX_SEGMENTS = 1 << 20;   // n_atoms * n_species accepted by the entry point
constexpr size_t NOALLOC_COUNT_BYTES = ((sizeof(int32_t) * (NOALLOC_MAX_SEGMENTS + 1) + 255) / 256) * 256;
constexpr size_t NOALLOC_SCAN_ITEMS = NOALLOC_MAX_SEGMENTS / SCAN_TILE + 3;
constexpr size_t NOALLOC_BYTES = NOALLOC_COUNT_BYTES + sizeof(int64_t) * NOALLOC_SCAN_ITEMS;   // about 4 MiB

static __device__ __align__(256) unsigned char g_export_scratch[NOALLOC_BYTES];

// In host code `g_export_scratch` is only a handle for the runtime, not a device address; the
// address a kernel may use comes from cudaGetSymbolAddress, asked once per device with that device
// current.  Slot d caches device d's answer.  The cache is plain host state: fill it from one host thread at a time,
// and a cudaDeviceReset() of that device invalidates the cached address (the library is not meant to outlive one).
static void *g_export_scratch_addr[64] = {nullptr};

static int export_scratch_for_current_device(mlip_ctx *c, void **out) {
    int dev = -1;
    MLIP_CUDA_TRY(c, cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) { c->err = "device ordinal out of range for the static scratch table"; return MLIP_ERR_UNSUPPORTED; }
    if (!g_export_scratch_addr[dev]) {
        void *p = nullptr;
        MLIP_CUDA_TRY(c, cudaGetSymbolAddress(&p, g_export_scratch));
        g_export_scratch_addr[dev] = p;
    }
    *out = g_export_scratch_addr[dev];
    return MLIP_OK;
}

// Same kernels and the same order as launch_export, with the temporaries taken from the static
// array.  Every scratch word that is read (counts of all n * C segments, the scan's tile sums) is
// written earlier in the same call, so nothing has to be cleared between calls; two calls whose
// kernels overlap on the GPU (different streams or contexts on one device) would race on it.
int launch_export_noalloc(mlip_ctx *c, int64_t *seg_ptr, int32_t *nbr, int64_t capacity, int64_t *n_entries_host, cudaStream_t s) {
    const int64_t n = c->n;
    const int C = c->cfg.n_species;
    if (n * C > NOALLOC_MAX_SEGMENTS) {
        c->err = "mlip_get_neighbors_noalloc: n_atoms * n_species exceeds 1048576 (the static scratch size); use mlip_get_neighbors";
        return MLIP_ERR_UNSUPPORTED;
    }
    void *base = nullptr;
    int rc = lists_whole(c, s);
    if (rc != MLIP_OK) return rc;
    if ((rc = export_scratch_for_current_device(c, &base)) != MLIP_OK) return rc;
    int32_t *seg_count = reinterpret_cast<int32_t *>(base);
    int64_t *tmp = reinterpret_cast<int64_t *>(static_cast<unsigned char *>(base) + NOALLOC_COUNT_BYTES);
    k_export_count<<<blocks_for(n * 32, 256), 256, 0, s>>>(n, C, c->nbr_off, list_view(c), c->pos4, c->user_of, seg_count);
    exclusive_scan<int32_t, int64_t>(seg_count, seg_ptr, n * C, tmp, s);
    MLIP_CUDA_TRY(c, cudaMemcpyAsync(c->total_host, seg_ptr + n * C, sizeof(int64_t), cudaMemcpyDeviceToHost, s));
    MLIP_CUDA_TRY(c, cudaStreamSynchronize(s));
    c->launches += 4;
    if (n_entries_host) *n_entries_host = *c->total_host;
    if (*c->total_host > capacity || !nbr) {
        c->err = "neighbor export: capacity too small";
        return MLIP_ERR_NEIGHBOR_OVERFLOW;
    }
    k_export_fill<<<blocks_for(n * 32, 256), 256, 0, s>>>(n, C, c->nbr_off, list_view(c), c->pos4, c->user_of, seg_ptr, nbr);
    c->launches += 1;
    MLIP_CUDA_TRY(c, cudaStreamSynchronize(s));
    return MLIP_OK;
}

}  // namespace mlip
