// The fused evaluation kernel (Section 3.4.1 "mega-fusion": Eq. 1-10 in one launch; every
// per-pair and per-atom intermediate lives in registers or shared memory, and the radial and
// angular features are recomputed in the derivation stage instead of being kept).
//
// Work decomposition
//   One persistent CTA of 16 warps per SM, organised as two independent groups of 8 warps.  The CTA
//   walks through the central species in order; for each it stages that species' radial tables
//   (one per neighbor species) and head constants in shared memory, then each group takes tiles of
//   8 central atoms of that species from a global counter (warp = atom) and runs them on its own,
//   synchronising only inside the group (named barriers), so that one group's latency-bound head
//   overlaps the other group's pair loops.
//   Encoding    The warp scans the atom's list (lane = entry), queues the pairs inside r_cut in
//               shared memory, and every 32 queued pairs evaluates harmonics (Eq. 3) and the
//               spline basis with lane = pair.  The moment P_i = H^T G (Eq. 4, 16 x n times
//               n x 32) is accumulated on the tensor pipe: mma.sync m16n8k8 TF32 with a
//               three-term hi/lo split of both operands (~2^-21 relative, fp32 accumulate), the
//               radial values g being evaluated straight into the B fragments.  P_i stays in
//               the accumulator registers until the derivation.
//   Invariants  Eq. 5 from the accumulator fragments by three xor-shuffles.
//   Regression  Eq. 6 forward and reverse for the 8 atoms of the tile at once as W X^T on the tensor
//               pipe (weights pre-packed in A-fragment order, 2-way split over the reduction
//               dimension across the group's warps, elementwise epilogue over the group's threads).
//               The current species' weights live in tensor memory (tcgen05.alloc / st / ld): a warp
//               fetches the 32 registers of its next contraction in one instruction, off the
//               L1/shared-memory pipe; the hidden layers are stored already split into hi + lo.
//   Derivation  W_i (Eq. 7) is the accumulator fragment of P_i scaled in place: by construction
//               of the channel permutation it already is the B fragment of the next contraction.
//               [V; T] = [G; G'] W^T (Eq. 9 and the re-associated Eq. 8 term, U_i never formed)
//               on the tensor pipe, 16 pairs per tile; results are transposed through shared
//               memory to lane = pair for the projection of Eq. 10 and the scatter.
// Everything that is not a contraction (geometry, harmonics, splines, projection) stays on the
// fp32 pipe; positions are differenced in fp64.
// Lists come in two parts (neighbor.cu): entries that were within r_cut + skin / 2 at build time first, the rest
// behind them; the far part cannot reach r_cut before some atom has moved skin / 4, and is skipped until the
// integrator raises far_flag.
// Operand splits for the three-term TF32 products are packed fp32 arithmetic (two values per instruction): a
// Veltkamp split where the result feeds energies, a truncating split where it feeds forces only.
#include <algorithm>

#include "common.cuh"
#include "pair_math.cuh"

namespace mlip {

constexpr int TILE = 8;       // atoms per tile = warps per group
constexpr int NG = 2;         // groups per CTA
constexpr int NW = NG * TILE; // warps per CTA
constexpr int PB_CAP = 160;   // queued pairs per warp: up to 31 left over + four list chunks of 32
constexpr int J_BITS = 28;    // queue entries pack the neighbor index (low 28 bits) with its species
constexpr int ST_STRIDE = 24; // encoding hand-over: 16 h, 4 b, table offset (bank-conflict-free for the fragment reads)
constexpr int BS_STRIDE = 12; // derivation hand-over: 4 b, 4 b', table offset
constexpr int VT_STRIDE = 40; // 16 v + 16 t per pair
constexpr int X_STRIDE = 132; // invariants / dE/dG per atom
constexpr int Z_STRIDE = 68;  // head activations per atom
#ifndef MLIP_TAB_STRIDE
#define MLIP_TAB_STRIDE 36
#endif
constexpr int TAB_STRIDE_SMEM = MLIP_TAB_STRIDE;   // padded table row in shared memory

constexpr int Q_WORDS = 4 * PB_CAP;                             // pair queue of a warp: kept from encoding to derivation
constexpr int SCR_WORDS = 32 * BS_STRIDE + 32 * VT_STRIDE;      // scratch of a warp: 384 + 1280
static_assert(32 * ST_STRIDE <= SCR_WORDS, "encoding stage must fit the derivation buffers");
constexpr int SX_WORDS = TILE * X_STRIDE;                       // per group
// head buffers of a group (alias of the scratch of the group's warps)
constexpr int HB_XS = 0;                                   // split invariants  [8][2 * X_STRIDE]
constexpr int HB_ZS = HB_XS + TILE * 2 * X_STRIDE;         // split activations [2][8][2 * Z_STRIDE]
constexpr int HB_DP = HB_ZS + 2 * TILE * 2 * Z_STRIDE;     // split dE/dpre     [8][2 * Z_STRIDE]
constexpr int HB_PART = HB_DP + TILE * 2 * Z_STRIDE;       // split-K partials  [2][8][Z_STRIDE]
constexpr int HB_WORDS = HB_PART + 2 * TILE * Z_STRIDE;
static_assert(HB_WORDS <= TILE * SCR_WORDS, "head buffers alias the scratch of the group's warps");
constexpr int HC_WORDS = HEAD_L * HEAD_H + HEAD_H + 16;         // biases, w_out, b_out of the current species
constexpr int64_t STAGGER_BELOW_ATOMS = 200000;                 // systems below this size start their CTAs on different species
constexpr int PF_IDX = 160;                                     // neighbor indices prefetched per warp for its next atom
constexpr int PF_CS = 96;                                       // compact lists: the codes take 81 words at most, the 27 cell bases sit here
static_assert(PF_IDX / 2 + 1 <= PF_CS && PF_CS + 27 <= PF_IDX, "prefetch buffer layout for compact lists");
constexpr int PF_WORDS = PF_IDX + 4;                            // + {atom, list start (2 words), list length}
constexpr int FIXED_WORDS = NG * SX_WORDS + NW * (Q_WORDS + SCR_WORDS + PF_WORDS) + HC_WORDS + 16;
constexpr int SMEM_LIMIT_WORDS = 227 * 1024 / 4 - 256;

// Pre-packed head weights per species (floats).  A record holds the A operand of one
// (m-tile, k-step): per lane {a0, a1, a2, a3}, i.e. 128 floats (split into hi + lo in registers).
//   forward  layer L: A[m][k] = W_L[m][k]   (m = neuron)    4 m-tiles, K_L / 8 k-steps
//   reverse  layer L: A[m][k] = W_L[k][m]   (m = input)     K_L / 16 m-tiles, 8 k-steps
// followed by biases [4][64], w_out[64], b_out, pad.
constexpr int KS0 = N_INV / 8, KS1 = HEAD_H / 8;
constexpr int FWD_RECORDS = 4 * KS0 + (HEAD_L - 1) * 4 * KS1;
constexpr int BWD_RECORDS = (N_INV / 16) * 8 + (HEAD_L - 1) * 4 * 8;
constexpr int HP_FWD = 0;
constexpr int HP_BWD = HP_FWD + FWD_RECORDS * 128;
constexpr int HP_BIAS = HP_BWD + BWD_RECORDS * 128;
constexpr int HP_WOUT = HP_BIAS + HEAD_L * HEAD_H;
constexpr int HP_TOTAL = HP_WOUT + HEAD_H + 4;

// SiLU and its derivative.  exp through the fast exponential: its error scales with |x| 2^-24 and
// enters the sigmoid damped by s (1 - s), far below fp32 rounding of the surrounding sums.
__device__ __forceinline__ float silu_f(float x, float &dsilu) {
    const float s = __fdividef(1.0f, 1.0f + __expf(-x));
    dsilu = s * (1.0f + x * (1.0f - s));
    return x * s;
}

// Two fp32 FMAs in one instruction (sm_100 packed arithmetic): d = a * b + c per component.  Halves the issue slots
// of the spline evaluations, whose operands already sit in register pairs from 128-bit loads.
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
    unsigned long long ra, rb, rc, rd;
    asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(a.x), "f"(a.y));
    asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(b.x), "f"(b.y));
    asm("mov.b64 %0, {%1, %2};" : "=l"(rc) : "f"(c.x), "f"(c.y));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(rd) : "l"(ra), "l"(rb), "l"(rc));
    float2 d;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d.x), "=f"(d.y) : "l"(rd));
    return d;
}

__device__ __forceinline__ void split_tf32(float x, uint32_t &hi, uint32_t &lo) {
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(hi) : "f"(x));
    lo = __float_as_uint(x - __uint_as_float(hi));
}
__device__ __forceinline__ float2 split_pair(float x) {
    uint32_t hi, lo;
    split_tf32(x, hi, lo);
    return make_float2(__uint_as_float(hi), __uint_as_float(lo));
}

// Two-at-a-time variant for operands that feed forces only.  The tensor pipe reads the upper 19 bits of a TF32 operand
// and ignores the rest, so the fp32 value itself serves as "hi" (= its truncation) and lo = x - trunc(x), taken for two
// values by one packed subtract: 1.5 instructions per value instead of 2, at one bit less in the lo term.
__device__ __forceinline__ float2 sub2(float2 a, float2 b) {
    unsigned long long ra, rb, rd;
    asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(a.x), "f"(a.y));
    asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(b.x), "f"(b.y));
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(rd) : "l"(ra), "l"(rb));
    float2 d;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d.x), "=f"(d.y) : "l"(rd));
    return d;
}
__device__ __forceinline__ float2 add2(float2 a, float2 b) {
    unsigned long long ra, rb, rd;
    asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(a.x), "f"(a.y));
    asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(b.x), "f"(b.y));
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(rd) : "l"(ra), "l"(rb));
    float2 d;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d.x), "=f"(d.y) : "l"(rd));
    return d;
}
// Rounded hi/lo split of two values in four packed fp32 operations (Veltkamp's splitting with the constant 2^13 + 1:
// hi keeps 11 significant bits, rounded to nearest, so it is exact in TF32; lo = x - hi exactly).  Same result as
// split_tf32 up to ties, but on the FMA pipe and two values at a time -- the conversion instruction expands into integer
// operations on the half-rate pipe.  For the energy path, where the truncating split's bias would show.
// The product is written as an explicit fused multiply-add with a zero addend: given a separate packed multiply, the
// assembler contracts it with the subtraction that follows (even with .rn on both), which turns the split into hi = x.
__device__ __forceinline__ void split2_rn(float x, float y, uint32_t &xh, uint32_t &yh, uint32_t &xl, uint32_t &yl) {
    const float2 v = make_float2(x, y);
    const float2 c = ffma2(v, make_float2(8193.f, 8193.f), make_float2(0.f, 0.f));
    const float2 hi = sub2(c, sub2(c, v));
    const float2 lo = sub2(v, hi);
    xh = __float_as_uint(hi.x); yh = __float_as_uint(hi.y); xl = __float_as_uint(lo.x); yl = __float_as_uint(lo.y);
}
__device__ __forceinline__ void split2_force(float x, float y, uint32_t &xh, uint32_t &yh, uint32_t &xl, uint32_t &yl) {
    xh = __float_as_uint(x); yh = __float_as_uint(y);
    const float2 lo = sub2(make_float2(x, y), make_float2(__uint_as_float(xh & 0xffffe000u), __uint_as_float(yh & 0xffffe000u)));
    xl = __float_as_uint(lo.x); yl = __float_as_uint(lo.y);
}

__device__ __forceinline__ void mma_tf32(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// d = A B (zero accumulator input: saves initialising the accumulator registers)
__device__ __forceinline__ void mma_tf32_z(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}

// Every product A B below has both operands split: A_hi B_hi + A_lo B_hi + A_hi B_lo.  The tensor
// pipe truncates when it adds into its fp32 accumulator, so the energy path keeps accumulation
// chains short (a fresh accumulator per k-step, folded into the running sum by a rounded fp32
// add): a long chain of same-sign terms otherwise drifts by ~1e-6 relative.

// Deterministic mode (force_mode = 1): every sum whose order depends on scheduling -- the force scatter across
// warps, the energy and virial totals -- is taken in integer arithmetic, which is associative, so two runs on the
// same input agree bit for bit.  Per-atom and per-pair terms are computed in a fixed order in either mode.
constexpr float FORCE_FX = 4294967296.f;        // 2^32 per eV/Angstrom
constexpr double ENERGY_FX = 4294967296.0;      // 2^32 per eV
constexpr double VIRIAL_FX = 268435456.0;       // 2^28 per eV
__device__ __forceinline__ void fixed_add3(long long *p, float x, float y, float z) {
    atomicAdd(reinterpret_cast<unsigned long long *>(p), (unsigned long long)__float2ll_rn(x * FORCE_FX));
    atomicAdd(reinterpret_cast<unsigned long long *>(p + 1), (unsigned long long)__float2ll_rn(y * FORCE_FX));
    atomicAdd(reinterpret_cast<unsigned long long *>(p + 2), (unsigned long long)__float2ll_rn(z * FORCE_FX));
}

struct KernelArgs {
    int64_t n;
    int n_species;
    CellGrid grid;
    double rc2;
    TableDesc tab;
    const double4 *pos4;
    const int32_t *center_order;
    const int32_t *species_start;
    const int64_t *nbr_off;
    const int32_t *nbr_near;   // leading entries of each list that can be inside r_cut while far_flag is down
    const int *far_flag;
    const int32_t *nbr;
    const uint16_t *nbr16;     // the same array when the lists hold 16-bit cell-relative codes (L16 instantiations)
    const int32_t *cell_id;    // build-time cell of each atom (L16)
    const int32_t *cell_start; // first atom of each cell (L16)
    int64_t nbr_cap;           // entries the list array holds (range-checked builds)
    const float *head_pack;
    float4 *force;
    long long *force_fx;   // deterministic mode: forces as 2^-32 eV/Angstrom integers [N][3]
    long long *acc_fx;     // deterministic mode: energy (2^-32 eV) and virial (2^-28 eV) integers [10]
    float *e_atom;
    double *acc;
    unsigned long long *pair_counter;
    int *status;
    int *tile_counter;
};

// One 256-bit load per gathered atom (a 32-byte sector) instead of two 128-bit ones: halves the
// number of L1 wavefronts of the uncoalesced position gathers.
__device__ __forceinline__ double4 load_pos4(const double4 *p) {
    double4 v;
    asm volatile("ld.global.nc.v4.f64 {%0,%1,%2,%3}, [%4];" : "=d"(v.x), "=d"(v.y), "=d"(v.z), "=d"(v.w) : "l"(p));
    return v;
}

// Where the radial tables of the current central species live: shared memory (rows padded to
// TAB_STRIDE_SMEM, table index = neighbor species) or, when they do not fit, global memory.
struct TableView {
    const float *base;
    int row_stride;     // floats per row
    int table_stride;   // floats per neighbor species
};

// Fill the warp's pair queue from list position `cur` on (lane = entry), up to five 32-entry chunks
// at a time with all index loads, then all position gathers, in flight together (a typical list
// of ~134 entries is one round trip).  Pairs inside r_cut are queued as {x, y, z, j | species << 28}.
// Stops when the list ends or the next group might not fit; returns the number of queued pairs
// and advances `cur`.  The first n_pref indices of the list may come from shared memory (sidx).
constexpr int SCAN_CHUNKS = 5;
static_assert(SCAN_CHUNKS * 32 <= PB_CAP, "a full group must fit an empty queue");
// Compact lists: lane q < 27 holds the first atom of the q-th cell around atom i's build-time cell; an entry's index is
// that base (one shuffle) plus the position coded in its low bits.
__device__ __forceinline__ int cell_base_of_lane(const KernelArgs &k, int i, int lane) {
    return lane < 27 ? __ldg(k.cell_start + neighbor_cell(k.grid, __ldg(k.cell_id + i), lane)) : 0;
}
template <int SCAN_CHUNKS, bool L16>
__device__ __forceinline__ int collect_pairs_n(const KernelArgs &k, const double4 &pi, int64_t beg, int64_t &cur, int64_t end, float4 *pq, int lane,
                                               const int *sidx, int n_pref, int cs) {
    int nq = 0;
    while (cur < end && nq + (int)min((int64_t)(SCAN_CHUNKS * 32), end - cur) <= PB_CAP) {
        int jj[SCAN_CHUNKS];
#pragma unroll
        for (int c = 0; c < SCAN_CHUNKS; ++c) {
            const int64_t e = cur + 32 * c + lane;
            if (L16) {   // (the prefetch copied whole 32-bit words starting at the even entry at or before `beg`)
                const int code = e < end ? (e - beg < n_pref ? reinterpret_cast<const uint16_t *>(sidx)[(e - beg) + (beg & 1)]
                                                             : __ldg(k.nbr16 + MLIP_CHECK_INDEX(e, k.nbr_cap, k.status))) : 0;
                const int base = __shfl_sync(0xffffffffu, cs, code >> L16_SHIFT);
                jj[c] = e < end ? base + (code & L16_MASK) : -1;
            } else {
                jj[c] = e < end ? (e - beg < n_pref ? sidx[e - beg] : __ldg(k.nbr + MLIP_CHECK_INDEX(e, k.nbr_cap, k.status))) : -1;
            }
            if (jj[c] >= 0) jj[c] = (int)MLIP_CHECK_INDEX(jj[c], k.n, k.status);
        }
        double4 pp[SCAN_CHUNKS];
#pragma unroll
        for (int c = 0; c < SCAN_CHUNKS; ++c) pp[c] = load_pos4(k.pos4 + (jj[c] < 0 ? 0 : jj[c]));
#pragma unroll
        for (int c = 0; c < SCAN_CHUNKS; ++c) {
            if (cur + 32 * c >= end) continue;   // warp-uniform: nothing in this chunk
            const double dx = min_image(pp[c].x - pi.x, k.grid.box[0], k.grid.half[0]);
            const double dy = min_image(pp[c].y - pi.y, k.grid.box[1], k.grid.half[1]);
            const double dz = min_image(pp[c].z - pi.z, k.grid.box[2], k.grid.half[2]);
            const double d2 = dx * dx + dy * dy + dz * dz;
            const bool valid = jj[c] >= 0 && d2 < k.rc2;
            const unsigned m = __ballot_sync(0xffffffffu, valid);
            if (valid)
                pq[nq + __popc(m & ((1u << lane) - 1u))] =
                    make_float4((float)dx, (float)dy, (float)dz, __int_as_float(jj[c] | ((int)pp[c].w << J_BITS)));
            nq += __popc(m);
        }
        cur += SCAN_CHUNKS * 32;
    }
    __syncwarp();
    return nq;
}
// Short lists (the usual case while the far entries are skipped) take the three-chunk form: fewer loads in flight,
// fewer registers.
template <bool L16>
__device__ __forceinline__ int collect_pairs(const KernelArgs &k, const double4 &pi, int64_t beg, int64_t &cur, int64_t end, float4 *pq, int lane,
                                             const int *sidx, int n_pref, int cs) {
    if (end - beg <= 96) return collect_pairs_n<3, L16>(k, pi, beg, cur, end, pq, lane, sidx, n_pref, cs);
    return collect_pairs_n<5, L16>(k, pi, beg, cur, end, pq, lane, sidx, n_pref, cs);
}

// ---------------- Encoding of one atom: returns the moment as accumulator fragments ----------------
// `queued` returns the number of pairs left in the queue when the whole list fitted in one round
// (the derivation then reuses them), or -1.
template <bool TAB_SMEM, bool L16>
__device__ __forceinline__ int encode_atom(const KernelArgs &k, const TableView &tv, const double4 &pi, int64_t beg, int64_t end,
                                           float4 *pq, float *stage, int lane, float (&Pf)[4][4], int &queued, const int *sidx, int n_pref,
                                           int cs, PhaseClock &pc) {
    const int g = lane >> 2, t = lane & 3;
    constexpr int rs = TAB_SMEM ? TAB_STRIDE_SMEM : K_RADIAL;   // = tv.row_stride, known here so that row offsets fold into the loads
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) Pf[a][b] = 0.f;

    auto batch = [&](int first, int n) {
        {   // lane = pair: harmonics (Eq. 3) and spline basis
            float h[D_ANG], b[4];
            int off = 0;
            if (lane < n) {
                const float4 e = pq[first + lane];
                const float d2 = e.x * e.x + e.y * e.y + e.z * e.z, rinv = rsqrtf(d2), r = d2 * rinv;
                harmonics(e.x * rinv, e.y * rinv, e.z * rinv, h);
                const int iv = spline_basis<false, float>(r, k.tab.r_min, k.tab.inv_h, k.tab.knots, b, nullptr, k.status);
                const int sj = __float_as_int(e.w) >> J_BITS;
                off = sj * tv.table_stride + iv * rs;
            } else {
#pragma unroll
                for (int a = 0; a < D_ANG; ++a) h[a] = 0.f;
                b[0] = b[1] = b[2] = b[3] = 0.f;
            }
            // 16-byte chunk c of row r is stored at chunk c ^ ((r >> 2) & 1): the eight rows of a store phase
            // then fall into eight different bank groups (the row stride alone gives only four)
            const int sw = (lane >> 2) & 1;
            float4 *row = reinterpret_cast<float4 *>(stage + lane * ST_STRIDE);
            row[0 ^ sw] = make_float4(h[0], h[1], h[2], h[3]);
            row[1 ^ sw] = make_float4(h[4], h[5], h[6], h[7]);
            row[2 ^ sw] = make_float4(h[8], h[9], h[10], h[11]);
            row[3 ^ sw] = make_float4(h[12], h[13], h[14], h[15]);
            row[4 ^ sw] = make_float4(b[0], b[1], b[2], b[3]);
            reinterpret_cast<int *>(stage)[lane * ST_STRIDE + 4 * (5 ^ sw)] = off;
        }
        __syncwarp();
        pc.mark(1);
        const int nks = (n + 7) >> 3;
#ifndef MLIP_KSTEP_UNROLL
#define MLIP_KSTEP_UNROLL 4
#endif
        constexpr int kstep_unroll = MLIP_KSTEP_UNROLL;
#pragma unroll kstep_unroll
        for (int ks = 0; ks < nks; ++ks) {
            // A = H^T (16 x 8 pairs): rows a = g, g + 8; columns pairs t, t + 4 of this k-step
            const float *ra = stage + (8 * ks + t) * ST_STRIDE, *rb = ra + 4 * ST_STRIDE;
            uint32_t ah[4], al[4];
            split2_rn(ra[g], ra[g + 8], ah[0], ah[1], al[0], al[1]);
            split2_rn(rb[g ^ 4], rb[(g ^ 4) + 8], ah[2], ah[3], al[2], al[3]);   // rows t + 4 are stored with their chunk pairs swapped
            // B = G (8 pairs x 8 channels per n-tile).  Evaluation pattern: quarter-warp q reads the table
            // rows of ONE pair (8 lanes x 16 bytes = a full row per access: no bank conflicts), i.e. lane
            // (q, c) evaluates channels 4c .. 4c+3 of pairs q and q + 4 of this k-step; a fixed shuffle
            // then hands the values to the lane that owns them in the B fragment (pair t, channels 4g .. 4g+3).
            const int q = lane >> 3, cch = lane & 7;
            const float *qa = stage + (8 * ks + q) * ST_STRIDE, *qb = qa + 4 * ST_STRIDE;
            const float4 ba = *reinterpret_cast<const float4 *>(qa + 16), bb = *reinterpret_cast<const float4 *>(qb + 20);
            const float *ta = tv.base + reinterpret_cast<const int *>(qa)[20] + 4 * cch;
            const float *tb = tv.base + reinterpret_cast<const int *>(qb)[16] + 4 * cch;
            const float4 a0 = *reinterpret_cast<const float4 *>(ta), a1 = *reinterpret_cast<const float4 *>(ta + rs);
            const float4 a2 = *reinterpret_cast<const float4 *>(ta + 2 * rs), a3 = *reinterpret_cast<const float4 *>(ta + 3 * rs);
            const float4 b0 = *reinterpret_cast<const float4 *>(tb), b1 = *reinterpret_cast<const float4 *>(tb + rs);
            const float4 b2 = *reinterpret_cast<const float4 *>(tb + 2 * rs), b3 = *reinterpret_cast<const float4 *>(tb + 3 * rs);
            float ga[4], gb[4];
            {   // g = sum_m b_m c_m for the four channels of each pair, two channels per packed FMA
                float2 lo, hi;
                lo = ffma2(make_float2(ba.x, ba.x), make_float2(a0.x, a0.y), make_float2(0.f, 0.f));
                hi = ffma2(make_float2(ba.x, ba.x), make_float2(a0.z, a0.w), make_float2(0.f, 0.f));
                lo = ffma2(make_float2(ba.y, ba.y), make_float2(a1.x, a1.y), lo);
                hi = ffma2(make_float2(ba.y, ba.y), make_float2(a1.z, a1.w), hi);
                lo = ffma2(make_float2(ba.z, ba.z), make_float2(a2.x, a2.y), lo);
                hi = ffma2(make_float2(ba.z, ba.z), make_float2(a2.z, a2.w), hi);
                lo = ffma2(make_float2(ba.w, ba.w), make_float2(a3.x, a3.y), lo);
                hi = ffma2(make_float2(ba.w, ba.w), make_float2(a3.z, a3.w), hi);
                ga[0] = lo.x; ga[1] = lo.y; ga[2] = hi.x; ga[3] = hi.y;
                lo = ffma2(make_float2(bb.x, bb.x), make_float2(b0.x, b0.y), make_float2(0.f, 0.f));
                hi = ffma2(make_float2(bb.x, bb.x), make_float2(b0.z, b0.w), make_float2(0.f, 0.f));
                lo = ffma2(make_float2(bb.y, bb.y), make_float2(b1.x, b1.y), lo);
                hi = ffma2(make_float2(bb.y, bb.y), make_float2(b1.z, b1.w), hi);
                lo = ffma2(make_float2(bb.z, bb.z), make_float2(b2.x, b2.y), lo);
                hi = ffma2(make_float2(bb.z, bb.z), make_float2(b2.z, b2.w), hi);
                lo = ffma2(make_float2(bb.w, bb.w), make_float2(b3.x, b3.y), lo);
                hi = ffma2(make_float2(bb.w, bb.w), make_float2(b3.z, b3.w), hi);
                gb[0] = lo.x; gb[1] = lo.y; gb[2] = hi.x; gb[3] = hi.y;
            }
            const int owner_src = 8 * t + g;   // lane (g, t) takes (pair t, chunk g) from lane (q = t, c = g)
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                ga[nt] = __shfl_sync(0xffffffffu, ga[nt], owner_src);
                gb[nt] = __shfl_sync(0xffffffffu, gb[nt], owner_src);
            }
            // Eq. 4 for eight pairs; the three terms of each n-tile are issued interleaved over the n-tiles
            uint32_t bh[4][2], bl[4][2];
            float c[4][4];
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) split2_rn(ga[nt], gb[nt], bh[nt][0], bh[nt][1], bl[nt][0], bl[nt][1]);
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) mma_tf32_z(c[nt], al[0], al[1], al[2], al[3], bh[nt][0], bh[nt][1]);
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) mma_tf32(c[nt], ah[0], ah[1], ah[2], ah[3], bl[nt][0], bl[nt][1]);
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) mma_tf32(c[nt], ah[0], ah[1], ah[2], ah[3], bh[nt][0], bh[nt][1]);
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                const float2 s01 = add2(make_float2(Pf[nt][0], Pf[nt][1]), make_float2(c[nt][0], c[nt][1]));
                const float2 s23 = add2(make_float2(Pf[nt][2], Pf[nt][3]), make_float2(c[nt][2], c[nt][3]));
                Pf[nt][0] = s01.x; Pf[nt][1] = s01.y; Pf[nt][2] = s23.x; Pf[nt][3] = s23.y;
            }
        }
        __syncwarp();
        pc.mark(2);
    };
    int total = 0, rounds = 0, n = 0;
    int64_t cur = beg;
    do {
        n = collect_pairs<L16>(k, pi, beg, cur, end, pq, lane, sidx, n_pref, cs);
        pc.mark(0);
        for (int q0 = 0; q0 < n; q0 += 32) batch(q0, min(32, n - q0));
        total += n;
        ++rounds;
    } while (cur < end);
    queued = rounds == 1 ? n : -1;
    return total;
}

// ---------------- Derivation of one atom (Eq. 8-10) ----------------
template <bool TAB_SMEM, bool DET, bool L16>
__device__ __forceinline__ void derive_atom(const KernelArgs &k, const TableView &tv, int i,
                                            float4 *pq, float *scr, int queued, int lane, const uint32_t (&Wh)[4][4],
                                            const uint32_t (&Wl)[4][4], float (&vir)[9], PhaseClock &pc) {
    const int g = lane >> 2, t = lane & 3;
    float *bs = scr, *vt = scr + 32 * BS_STRIDE;
    constexpr int rs = TAB_SMEM ? TAB_STRIDE_SMEM : K_RADIAL;
    float fx = 0.f, fy = 0.f, fz = 0.f;

    auto batch = [&](int first, int n) {
        {   // lane = pair: spline basis and its derivative
            float4 ent = make_float4(1.f, 0.f, 0.f, 0.f);
            float b[4] = {0.f, 0.f, 0.f, 0.f}, db[4] = {0.f, 0.f, 0.f, 0.f};
            int off = 0, row_index = 0;
            const bool live = lane < n;
            if (live) {
                ent = pq[first + lane];
                const float d2 = ent.x * ent.x + ent.y * ent.y + ent.z * ent.z, r = d2 * rsqrtf(d2);
                const int iv = spline_basis<true, float>(r, k.tab.r_min, k.tab.inv_h, k.tab.knots, b, db, k.status);
                row_index = (__float_as_int(ent.w) >> J_BITS) * (k.tab.knots + 3) + iv;
                off = row_index * rs;
            }
            const int slot = lane;
            float4 *row = reinterpret_cast<float4 *>(bs + slot * BS_STRIDE);
            row[0] = make_float4(b[0], b[1], b[2], b[3]);
            row[1] = make_float4(db[0], db[1], db[2], db[3]);
            reinterpret_cast<int *>(bs)[slot * BS_STRIDE + 8] = off;
            // geometry for the projection, which runs with lane = slot (spare chunk of the V/T row; the row's
            // 16-byte chunks are stored at chunk ^ ((slot >> 2) & 1) so that lane = row reads hit eight bank groups)
            *reinterpret_cast<float4 *>(vt + slot * VT_STRIDE + 32 + 4 * ((slot >> 2) & 1)) = ent;
        }
        __syncwarp();
        pc.mark(4);
        const int nmt = (n + 15) >> 4;
#ifndef MLIP_MTILE_UNROLL
#define MLIP_MTILE_UNROLL 1
#endif
        constexpr int mtile_unroll = MLIP_MTILE_UNROLL;
#pragma unroll mtile_unroll
        for (int mt = 0; mt < nmt; ++mt) {
            // A = [G; G'] (16 pairs x 32 channels): rows pairs g, g + 8; this lane evaluates channels 8t .. 8t+7
            // (one accumulator per output here: the truncating accumulation costs ~1e-6 relative on a
            // 12-term chain, irrelevant for forces, and the registers are needed elsewhere)
            float V[2][4], T[2][4];
            float G[2][8], dG[2][8];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const float *rp = bs + (16 * mt + g + 8 * q) * BS_STRIDE;
                const float4 b = *reinterpret_cast<const float4 *>(rp), db = *reinterpret_cast<const float4 *>(rp + 4);
                const float *tc = tv.base + reinterpret_cast<const int *>(rp)[8] + 8 * t;
                const float bw[4] = {b.x, b.y, b.z, b.w}, dbw[4] = {db.x, db.y, db.z, db.w};
                float2 G2[4], dG2[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) { G2[c] = make_float2(0.f, 0.f); dG2[c] = make_float2(0.f, 0.f); }
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    const float4 c0 = *reinterpret_cast<const float4 *>(tc + m * rs), c1 = *reinterpret_cast<const float4 *>(tc + m * rs + 4);
                    const float2 cv[4] = {make_float2(c0.x, c0.y), make_float2(c0.z, c0.w), make_float2(c1.x, c1.y), make_float2(c1.z, c1.w)};
                    const float2 b2 = make_float2(bw[m], bw[m]), db2 = make_float2(dbw[m], dbw[m]);
#pragma unroll
                    for (int c = 0; c < 4; ++c) { G2[c] = ffma2(b2, cv[c], G2[c]); dG2[c] = ffma2(db2, cv[c], dG2[c]); }
                }
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    G[q][2 * c] = G2[c].x; G[q][2 * c + 1] = G2[c].y;
                    dG[q][2 * c] = dG2[c].x; dG[q][2 * c + 1] = dG2[c].y;
                }
            }
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                uint32_t ah[4], al[4], dh[4], dl[4];
                split2_force(G[0][ks], G[1][ks], ah[0], ah[1], al[0], al[1]);
                split2_force(G[0][4 + ks], G[1][4 + ks], ah[2], ah[3], al[2], al[3]);
                split2_force(dG[0][ks], dG[1][ks], dh[0], dh[1], dl[0], dl[1]);
                split2_force(dG[0][4 + ks], dG[1][4 + ks], dh[2], dh[3], dl[2], dl[3]);
                // Eq. 9 (rows of V: a = 0..7 and 8..15) and W g' (Eq. 8 re-associated); cross terms first, the
                // four independent accumulators interleaved
                if (ks == 0) {
                    mma_tf32_z(V[0], al[0], al[1], al[2], al[3], Wh[ks][0], Wh[ks][1]);
                    mma_tf32_z(V[1], al[0], al[1], al[2], al[3], Wh[ks][2], Wh[ks][3]);
                    mma_tf32_z(T[0], dl[0], dl[1], dl[2], dl[3], Wh[ks][0], Wh[ks][1]);
                    mma_tf32_z(T[1], dl[0], dl[1], dl[2], dl[3], Wh[ks][2], Wh[ks][3]);
                } else {
                    mma_tf32(V[0], al[0], al[1], al[2], al[3], Wh[ks][0], Wh[ks][1]);
                    mma_tf32(V[1], al[0], al[1], al[2], al[3], Wh[ks][2], Wh[ks][3]);
                    mma_tf32(T[0], dl[0], dl[1], dl[2], dl[3], Wh[ks][0], Wh[ks][1]);
                    mma_tf32(T[1], dl[0], dl[1], dl[2], dl[3], Wh[ks][2], Wh[ks][3]);
                }
                mma_tf32(V[0], ah[0], ah[1], ah[2], ah[3], Wl[ks][0], Wl[ks][1]);
                mma_tf32(V[1], ah[0], ah[1], ah[2], ah[3], Wl[ks][2], Wl[ks][3]);
                mma_tf32(T[0], dh[0], dh[1], dh[2], dh[3], Wl[ks][0], Wl[ks][1]);
                mma_tf32(T[1], dh[0], dh[1], dh[2], dh[3], Wl[ks][2], Wl[ks][3]);
                mma_tf32(V[0], ah[0], ah[1], ah[2], ah[3], Wh[ks][0], Wh[ks][1]);
                mma_tf32(V[1], ah[0], ah[1], ah[2], ah[3], Wh[ks][2], Wh[ks][3]);
                mma_tf32(T[0], dh[0], dh[1], dh[2], dh[3], Wh[ks][0], Wh[ks][1]);
                mma_tf32(T[1], dh[0], dh[1], dh[2], dh[3], Wh[ks][2], Wh[ks][3]);
            }
            float *va = vt + (16 * mt + g) * VT_STRIDE + ((2 * t) ^ (g & 4)), *vb = va + 8 * VT_STRIDE;   // chunk ^ ((row >> 2) & 1)
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                *reinterpret_cast<float2 *>(va + 8 * q) = make_float2(V[q][0], V[q][1]);
                *reinterpret_cast<float2 *>(vb + 8 * q) = make_float2(V[q][2], V[q][3]);
                *reinterpret_cast<float2 *>(va + 16 + 8 * q) = make_float2(T[q][0], T[q][1]);
                *reinterpret_cast<float2 *>(vb + 16 + 8 * q) = make_float2(T[q][2], T[q][3]);
            }
        }
        __syncwarp();
        pc.mark(5);
        if (lane < n) {   // lane = pair: projection onto the pair vector (Eq. 10) and scatter
            float v[D_ANG], tt[D_ANG];
            const int sw = (lane >> 2) & 1;
            const float4 *src = reinterpret_cast<const float4 *>(vt + lane * VT_STRIDE);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float4 a = src[q ^ sw], b = src[(4 + q) ^ sw];
                v[4 * q] = a.x; v[4 * q + 1] = a.y; v[4 * q + 2] = a.z; v[4 * q + 3] = a.w;
                tt[4 * q] = b.x; tt[4 * q + 1] = b.y; tt[4 * q + 2] = b.z; tt[4 * q + 3] = b.w;
            }
            const float4 ent = src[8 ^ sw];
            const float x = ent.x, y = ent.y, z = ent.z;
            const float rinv = rsqrtf(x * x + y * y + z * z);
            const int j = __float_as_int(ent.w) & ((1 << J_BITS) - 1);
            const float ux = x * rinv, uy = y * rinv, uz = z * rinv;
            float s, tx, ty, tz, tu;
            harmonics_project(ux, uy, uz, v, tt, s, tx, ty, tz, tu);
            // f_ij = (g' . u_ij) r^ + J_ang^T v_ij,  J_ang = (grad_u h)(I - u u^T) / r
            const float qx = s * ux + (tx - tu * ux) * rinv;
            const float qy = s * uy + (ty - tu * uy) * rinv;
            const float qz = s * uz + (tz - tu * uz) * rinv;
            fx += qx; fy += qy; fz += qz;
            if (DET) fixed_add3(k.force_fx + 3 * (size_t)j, -qx, -qy, -qz);
            else atomicAdd(&k.force[j], make_float4(-qx, -qy, -qz, 0.f));   // one 128-bit reduction per pair
            vir[0] -= x * qx; vir[1] -= x * qy; vir[2] -= x * qz;
            vir[3] -= y * qx; vir[4] -= y * qy; vir[5] -= y * qz;
            vir[6] -= z * qx; vir[7] -= z * qy; vir[8] -= z * qz;
        }
        __syncwarp();
        pc.mark(6);
    };
    if (queued >= 0) {   // the encoding left every pair of this atom in the queue
        for (int q0 = 0; q0 < queued; q0 += 32) batch(q0, min(32, queued - q0));
    } else {   // rare: the list did not fit the queue; position and list bounds are fetched again rather than kept
               // in registers through the head
        const double4 pi = load_pos4(k.pos4 + i);
        const int64_t beg = k.nbr_off[i], end = *k.far_flag ? k.nbr_off[i + 1] : beg + k.nbr_near[i];
        int64_t cur = beg;
        const int cs = L16 ? cell_base_of_lane(k, i, lane) : 0;
        do {
            const int n = collect_pairs<L16>(k, pi, beg, cur, end, pq, lane, nullptr, 0, cs);
            pc.mark(3);
            for (int q0 = 0; q0 < n; q0 += 32) batch(q0, min(32, n - q0));
        } while (cur < end);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        fx += __shfl_xor_sync(0xffffffffu, fx, o);
        fy += __shfl_xor_sync(0xffffffffu, fy, o);
        fz += __shfl_xor_sync(0xffffffffu, fz, o);
    }
    if (lane == 0) {
        if (DET) fixed_add3(k.force_fx + 3 * (size_t)i, fx, fy, fz);
        else atomicAdd(&k.force[i], make_float4(fx, fy, fz, 0.f));
    }
}

// ---------------- Tensor memory (TMEM) as the home of the regression network's weights ----------------
// The SM's 256 KB of tensor memory (128 lanes x 512 columns of 32 bits) is otherwise idle in this kernel (the
// contractions are per-atom products too small for tcgen05.mma), and it is the one on-chip store large enough for a
// species' head: 41 k weights in MMA-fragment order for the forward and the reverse pass, 27 k of them with their hi/lo
// split already taken.  A warp reaches the 32 lanes of quarter (warp % 4); a "record" is one A fragment = 4 consecutive
// columns (a0..a3 of each lane).  The four warps of a quarter are the two roles (m-tile = quarter, k-half 0 / 1) of
// the two groups, so each role's region is written once per species (by group 0) and read by both groups.
//   region of role kh: columns 256 kh + ...
//     [  0,  32)  forward, first layer: 8 records as they are (split on the fly)
//     [ 32, 128)  forward, hidden layers 2-4: per layer 4 records hi, then 4 records lo (rounded split: energy path)
//     [128, 224)  reverse, hidden layers: per layer 4 records as they are, then 4 records lo of the truncating split
//     [224, 256)  reverse, first layer: 8 records as they are
// tcgen05.ld / st move 4, 16 or 32 consecutive columns between a thread's registers and its lane; they bypass the
// L1/shared-memory data pipe, which is this kernel's busiest unit.
constexpr uint32_t TM_COLS = 512;
constexpr int TM_ROLE = 256, TM_FWD0 = 0, TM_FWD = 32, TM_BWD = 128, TM_BWD0 = 224;

__device__ __forceinline__ void tmem_st4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t addr, uint32_t (&r)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
                   "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
                   "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
                   "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(addr) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// One warp of group 0 writes its role's region (wg = m-tile + 4 k-half) for the species whose packed weights start at hp.
__device__ __forceinline__ void tmem_fill_role(uint32_t region, const float *__restrict__ hp, int wg, int lane) {
    const float4 *fwd = reinterpret_cast<const float4 *>(hp + HP_FWD), *bwd = reinterpret_cast<const float4 *>(hp + HP_BWD);
    const int mt4 = wg & 3, kh = wg >> 2;
    auto as_is = [&](uint32_t col, const float4 *rec) {
        const float4 v = __ldg(rec + lane);
        tmem_st4(region + col, __float_as_uint(v.x), __float_as_uint(v.y), __float_as_uint(v.z), __float_as_uint(v.w));
    };
    // (the loops are unrolled so that a warp has 8 to 16 loads in flight: one L2 round trip per group of records instead of
    // one per record, which is what a small system's kernel time is made of)
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        as_is(TM_FWD0 + 4 * q, fwd + (size_t)(mt4 * KS0 + kh * 8 + q) * 32);
        as_is(TM_BWD0 + 4 * q, bwd + (size_t)(wg * 8 + q) * 32);
    }
#pragma unroll 1
    for (int b = 0; b < HEAD_L - 1; ++b)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            {   // forward: hi, lo of the rounded split
                const float4 v = __ldg(fwd + (size_t)(4 * KS0 + b * 4 * KS1 + mt4 * KS1 + kh * 4 + q) * 32 + lane);
                uint32_t h[4], l[4];
                split_tf32(v.x, h[0], l[0]); split_tf32(v.y, h[1], l[1]); split_tf32(v.z, h[2], l[2]); split_tf32(v.w, h[3], l[3]);
                tmem_st4(region + TM_FWD + 32 * b + 4 * q, h[0], h[1], h[2], h[3]);
                tmem_st4(region + TM_FWD + 32 * b + 16 + 4 * q, l[0], l[1], l[2], l[3]);
            }
            {   // reverse: the value itself (the tensor pipe truncates it), lo of the truncating split
                const float4 v = __ldg(bwd + (size_t)((N_INV / 16) * 8 + b * 32 + mt4 * 8 + kh * 4 + q) * 32 + lane);
                uint32_t h[4], l[4];
                split2_force(v.x, v.y, h[0], h[1], l[0], l[1]);
                split2_force(v.z, v.w, h[2], h[3], l[2], l[3]);
                tmem_st4(region + TM_BWD + 32 * b + 4 * q, h[0], h[1], h[2], h[3]);
                tmem_st4(region + TM_BWD + 32 * b + 16 + 4 * q, l[0], l[1], l[2], l[3]);
            }
        }
    tmem_wait_st();
}

// Barrier among the 256 threads of one group (hardware barrier 1 + group).
__device__ __forceinline__ void group_sync(int group) {
    asm volatile("bar.sync %0, %1;" ::"r"(group + 1), "r"(TILE * 32) : "memory");
}

// Head contraction on the tensor pipe: C^T[16 rows of W x 8 atoms] over NKS k-steps from ks0.
// A records come from tensor memory (32 columns = 8 records as stored, or 4 records hi + 4 records lo when PRE);
// B = activations (hi, lo interleaved) from shared memory with `bstride` floats per atom.
// FRESH: every k-step gets its own accumulator, folded in by a rounded add (energy path);
// otherwise one accumulation chain (reverse pass: feeds forces only).
template <int NKS, bool FRESH, bool PRE>
__device__ __forceinline__ void head_gemm(float (&c)[4], const uint32_t (&wr)[32], int ks0, const float *__restrict__ act, int bstride, int lane) {
    static_assert(NKS % 4 == 0, "k-steps are processed four at a time (four independent MMA chains in flight)");
    static_assert(!PRE || NKS == 4, "a pre-split load holds four records");
    const int g = lane >> 2, t = lane & 3;
    float acc[4][4];   // FRESH: per-k-step products; otherwise four accumulation chains
#pragma unroll
    for (int q = 0; q < NKS; q += 4) {
        uint32_t ah[4][4], al[4][4];
        float2 x0[4], x1[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float *r0 = act + g * bstride + 2 * (8 * (ks0 + q + u) + t);
            x0[u] = *reinterpret_cast<const float2 *>(r0);
            x1[u] = *reinterpret_cast<const float2 *>(r0 + 8);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int o = 4 * (q + u);
            if (PRE) {
#pragma unroll
                for (int e = 0; e < 4; ++e) { ah[u][e] = wr[o + e]; al[u][e] = wr[16 + o + e]; }
            } else if (FRESH) {
                split2_rn(__uint_as_float(wr[o]), __uint_as_float(wr[o + 1]), ah[u][0], ah[u][1], al[u][0], al[u][1]);
                split2_rn(__uint_as_float(wr[o + 2]), __uint_as_float(wr[o + 3]), ah[u][2], ah[u][3], al[u][2], al[u][3]);
            } else {
                split2_force(__uint_as_float(wr[o]), __uint_as_float(wr[o + 1]), ah[u][0], ah[u][1], al[u][0], al[u][1]);
                split2_force(__uint_as_float(wr[o + 2]), __uint_as_float(wr[o + 3]), ah[u][2], ah[u][3], al[u][2], al[u][3]);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (FRESH || q == 0) mma_tf32_z(acc[u], al[u][0], al[u][1], al[u][2], al[u][3], __float_as_uint(x0[u].x), __float_as_uint(x1[u].x));
            else mma_tf32(acc[u], al[u][0], al[u][1], al[u][2], al[u][3], __float_as_uint(x0[u].x), __float_as_uint(x1[u].x));
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) mma_tf32(acc[u], ah[u][0], ah[u][1], ah[u][2], ah[u][3], __float_as_uint(x0[u].y), __float_as_uint(x1[u].y));
#pragma unroll
        for (int u = 0; u < 4; ++u) mma_tf32(acc[u], ah[u][0], ah[u][1], ah[u][2], ah[u][3], __float_as_uint(x0[u].x), __float_as_uint(x1[u].x));
        if (FRESH) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float s4 = (acc[0][e] + acc[1][e]) + (acc[2][e] + acc[3][e]);
                c[e] = q == 0 ? s4 : c[e] + s4;
            }
        }
    }
    if (!FRESH) {
#pragma unroll
        for (int e = 0; e < 4; ++e) c[e] = (acc[0][e] + acc[1][e]) + (acc[2][e] + acc[3][e]);
    }
}

// c fragment (rows = 16 m + g, g + 8; columns = atoms 2t, 2t + 1) -> part[atom][row] with `pstride` floats per atom
__device__ __forceinline__ void store_partial(const float (&c)[4], float *part, int pstride, int m_tile, int lane) {
    const int g = lane >> 2, t = lane & 3;
    float *p = part + 2 * t * pstride + 16 * m_tile + g;
    p[0] = c[0]; p[pstride] = c[1]; p[8] = c[2]; p[pstride + 8] = c[3];
}

// Prefetch of the warp's atom in the group's NEXT tile, spread over three points of the head so
// that each dependent global load has a barrier's worth of time to arrive: centre index -> list
// bounds -> the first PF_IDX neighbor indices (cp.async straight into shared memory).  (Pulling the
// neighbors' positions into L2 as a fourth step cost more issue slots than it saved latency.)
struct NextAtom {
    const KernelArgs *k;
    int *meta;        // shared: {atom, list start lo, list start hi, list length}
    int *sidx;        // shared: neighbor indices
    int slot;         // position in center_order, or -1
    int i;
    bool use_far;     // the lists' far entries have to be scanned as well
    int64_t beg, end;
    int cid;          // compact lists: the atom's build-time cell
    __device__ __forceinline__ void stage_a() { if (slot >= 0) i = __ldg(k->center_order + slot); }
    template <bool L16>
    __device__ __forceinline__ void stage_b() {
        if (slot >= 0) {
            beg = __ldg(k->nbr_off + i); end = use_far ? __ldg(k->nbr_off + i + 1) : beg + __ldg(k->nbr_near + i);
            if (L16) cid = __ldg(k->cell_id + i);
        }
    }
    template <bool L16>
    __device__ __forceinline__ void stage_c(int lane) {
        if (slot < 0) return;
        const int n = (int)min((int64_t)PF_IDX, end - beg);
        if (L16) {   // codes travel as whole 32-bit words from the even entry at or before `beg`; the 27 cell bases follow them
            const int odd = (int)(beg & 1), words = (odd + n + 1) >> 1;
            const int *src = reinterpret_cast<const int *>(k->nbr16 + (beg - odd));
#pragma unroll
            for (int c = 0; c < (PF_IDX / 2 + 1 + 31) / 32; ++c) {
                const int e = 32 * c + lane;
                if (e < words) {
                    const unsigned dst = (unsigned)__cvta_generic_to_shared(sidx + e);
                    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src + e) : "memory");
                }
            }
            if (lane < 27) {
                const unsigned dst = (unsigned)__cvta_generic_to_shared(sidx + PF_CS + lane);
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(k->cell_start + neighbor_cell(k->grid, cid, lane)) : "memory");
            }
        } else {
#pragma unroll
            for (int c = 0; c < PF_IDX / 32; ++c) {
                const int e = 32 * c + lane;
                if (e < n) {
                    const unsigned dst = (unsigned)__cvta_generic_to_shared(sidx + e);
                    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(k->nbr + beg + e) : "memory");
                }
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        if (lane == 0) { meta[0] = i; meta[1] = (int)(beg & 0xffffffff); meta[2] = (int)(beg >> 32); meta[3] = (int)(end - beg); }
    }
};

// ---------------- Regression (Eq. 6) forward and reverse for the group's tile ----------------
// In: sX = invariants [atom][128].  Out: sX = dE/dG; per-atom energies written.
// hc = biases [4][64], w_out [64], b_out of the species in shared memory.  wg = warp within the group.
template <bool DET, bool L16>
__device__ __forceinline__ void head_tile(const KernelArgs &k, float *sX, float *hb, const float *hc, uint32_t tm_role, int count, int first,
                                          int group, int wg, int lane, double &e_sum, NextAtom &nx, PhaseClock &pc) {
    float *xs = hb + HB_XS, *zs = hb + HB_ZS, *dp = hb + HB_DP, *part = hb + HB_PART;
    const int mt4 = wg & 3, kh = wg >> 2;   // forward / reverse hidden layers: 4 m-tiles x 2 k-halves
    const int atom = wg;                    // elementwise phases: warp = atom, lane = neuron (and neuron + 32)
    uint32_t w[32];   // A records of the coming contraction, fetched from tensor memory just before it

    // split the invariants once
#pragma unroll
    for (int f = lane; f < N_INV; f += 64) {
        uint32_t h0, h1, l0, l1;
        split2_rn(sX[atom * X_STRIDE + f], sX[atom * X_STRIDE + f + 32], h0, h1, l0, l1);
        *reinterpret_cast<float2 *>(xs + atom * 2 * X_STRIDE + 2 * f) = make_float2(__uint_as_float(h0), __uint_as_float(l0));
        *reinterpret_cast<float2 *>(xs + atom * 2 * X_STRIDE + 2 * (f + 32)) = make_float2(__uint_as_float(h1), __uint_as_float(l1));
    }
    nx.stage_a();
    pc.mark(3);
    group_sync(group);
    pc.mark(14);

    float e_i = 0.f;
    float ya = 0.f, yb = 0.f;   // running activations of this thread's two neurons (the skip path)
    float2 dzn = make_float2(0.f, 0.f);   // dE/dy of the same two neurons in the reverse pass
    float2 sdr[HEAD_L];                    // SiLU' of their pre-activations, layer by layer
#pragma unroll
    for (int L = 0; L < HEAD_L; ++L) {
        const float *zin = zs + ((L + 1) & 1) * TILE * 2 * Z_STRIDE;
        float *zout = zs + (L & 1) * TILE * 2 * Z_STRIDE;
        float c[4];
        tmem_ld32(tm_role + (L == 0 ? TM_FWD0 : TM_FWD + 32 * (L - 1)), w);
        tmem_wait_ld();
        if (L == 0) head_gemm<KS0 / 2, true, false>(c, w, kh * (KS0 / 2), xs, 2 * X_STRIDE, lane);
        else head_gemm<KS1 / 2, true, true>(c, w, kh * (KS1 / 2), zin, 2 * Z_STRIDE, lane);
        pc.mark(12);
        store_partial(c, part + kh * TILE * Z_STRIDE, Z_STRIDE, mt4, lane);
        if (L == 0) nx.template stage_b<L16>();
        if (L == 1) nx.template stage_c<L16>(lane);
        pc.mark(13);
        group_sync(group);
        pc.mark(14);
        // elementwise: bias, SiLU, residual; this thread owns neurons 2 lane, 2 lane + 1 of its atom
        {
            const int n0 = 2 * lane;
            const float2 p0 = *reinterpret_cast<const float2 *>(part + atom * Z_STRIDE + n0);
            const float2 p1 = *reinterpret_cast<const float2 *>(part + (TILE + atom) * Z_STRIDE + n0);
            const float2 bb = *reinterpret_cast<const float2 *>(hc + L * HEAD_H + n0);
            float d0, d1;
            ya += silu_f((p0.x + p1.x) + bb.x, d0);
            yb += silu_f((p0.y + p1.y) + bb.y, d1);
            const float y0 = ya, y1 = yb;
            sdr[L] = make_float2(d0, d1);
            if (L < HEAD_L - 1) {
                uint32_t h0, h1, l0, l1;
                split2_rn(y0, y1, h0, h1, l0, l1);
                *reinterpret_cast<uint4 *>(zout + atom * 2 * Z_STRIDE + 2 * n0) = make_uint4(h0, l0, h1, l1);
            } else {   // output layer and the start of the reverse pass: dE/dz = w_out
                const float2 wo = *reinterpret_cast<const float2 *>(hc + HEAD_L * HEAD_H + n0);
                e_i += wo.x * y0 + wo.y * y1;
                dzn = wo;
                uint32_t h0, h1, l0, l1;
                split2_rn(wo.x * d0, wo.y * d1, h0, h1, l0, l1);
                *reinterpret_cast<uint4 *>(dp + atom * 2 * Z_STRIDE + 2 * n0) = make_uint4(h0, l0, h1, l1);
            }
        }
        pc.mark(15);
        group_sync(group);
        pc.mark(14);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) e_i += __shfl_xor_sync(0xffffffffu, e_i, o);
    e_i += hc[HEAD_L * HEAD_H + HEAD_H];
    if (lane == 0 && atom < count) {
        k.e_atom[__ldg(k.center_order + first + atom)] = e_i;
        e_sum += DET ? rint((double)e_i * ENERGY_FX) : (double)e_i;   // DET: exact integer sums
    }

    // reverse through the hidden layers 3, 2, 1 (each with its skip path)
#pragma unroll
    for (int L = HEAD_L - 1; L >= 1; --L) {
        float c[4];
        tmem_ld32(tm_role + TM_BWD + 32 * (L - 1), w);
        tmem_wait_ld();
        head_gemm<4, false, true>(c, w, kh * 4, dp, 2 * Z_STRIDE, lane);
        store_partial(c, part + kh * TILE * Z_STRIDE, Z_STRIDE, mt4, lane);
        group_sync(group);
        {
            const int n0 = 2 * lane;
            const float2 p0 = *reinterpret_cast<const float2 *>(part + atom * Z_STRIDE + n0);
            const float2 p1 = *reinterpret_cast<const float2 *>(part + (TILE + atom) * Z_STRIDE + n0);
            dzn.x += p0.x + p1.x; dzn.y += p0.y + p1.y;
            const float2 da = sdr[L - 1];
            uint32_t h0, h1, l0, l1;
            split2_rn(dzn.x * da.x, dzn.y * da.y, h0, h1, l0, l1);
            *reinterpret_cast<uint4 *>(dp + atom * 2 * Z_STRIDE + 2 * n0) = make_uint4(h0, l0, h1, l1);
        }
        group_sync(group);
    }
    {   // first layer: dE/dG [128 x 8], warp = m-tile (16 inputs), written over the invariants
        float c[4];
        tmem_ld32(tm_role + TM_BWD0, w);   // warp = m-tile, all 8 k-steps
        tmem_wait_ld();
        head_gemm<8, false, false>(c, w, 0, dp, 2 * Z_STRIDE, lane);
        store_partial(c, sX, X_STRIDE, wg, lane);
    }
    group_sync(group);
}

template <bool TAB_SMEM, bool DET, bool L16, bool STAGGER>
__global__ void __launch_bounds__(NW * 32, 1) k_mega(KernelArgs k, int tab_words) {
    extern __shared__ __align__(16) float smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int group = warp / TILE, wg = warp % TILE;
    const int g = lane >> 2, t = lane & 3;
    float *s_tab = smem;                                   // [C][rows][TAB_STRIDE_SMEM] when TAB_SMEM
    float *sX = smem + (TAB_SMEM ? tab_words : 0) + group * SX_WORDS;
    float *scr_all = smem + (TAB_SMEM ? tab_words : 0) + NG * SX_WORDS;
    float *hb = scr_all + group * TILE * SCR_WORDS;        // head buffers = the scratch of the group's warps
    float *scr = scr_all + warp * SCR_WORDS;
    float4 *pq = reinterpret_cast<float4 *>(scr_all + NW * SCR_WORDS + warp * Q_WORDS);
    int *pf = reinterpret_cast<int *>(scr_all + NW * (SCR_WORDS + Q_WORDS)) + warp * PF_WORDS;
    float *hc = scr_all + NW * (SCR_WORDS + Q_WORDS + PF_WORDS);
    int *ctl = reinterpret_cast<int *>(hc + HC_WORDS);
    const int rows = k.tab.knots + 3;
    // lists that an in-step rebuild could not complete (capacity, broken configuration) are not evaluated: the outputs
    // stay at their cleared values and the status word tells the caller why (nothing in this kernel raises these bits,
    // so every CTA takes the same decision)
    if (*k.status & (FLAG_NEIGHBOR_OVERFLOW | FLAG_NONFINITE)) return;
    const bool use_far = *k.far_flag != 0;   // an atom has moved skin / 4 since the build: every list entry counts

    // all of tensor memory (this is the only CTA on the SM) for the head's weights
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(ctl + 4)), "r"(TM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tmem_fence_before_sync();
    __syncthreads();
    tmem_fence_after_sync();
    const uint32_t tm_base = *reinterpret_cast<volatile uint32_t *>(ctl + 4);
    const uint32_t tm_role = tm_base + ((uint32_t)(32 * (wg & 3)) << 16) + TM_ROLE * (wg >> 2);

    double e_sum = 0.0;
    float vir[9] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    double vir_fx = 0.0;   // DET: lane q < 9 keeps component q as an exact integer-valued sum
    unsigned long long n_pairs = 0;
    TableView tv;
    PhaseClock pc;
    pc.start();

    // STAGGER (small systems): the CTAs start on different central species, so that the species are worked on side by
    // side rather than one after the other by mostly idle SMs (864 atoms: 64 instead of 92 us).  Large systems keep the
    // plain loop: one front through the cell-ordered atoms, and a loop counter as the species costs 1 % less than a
    // computed one.  Either way a species whose tiles are all claimed already is passed over: staging its tables would
    // be the only thing left to do.
    for (int ss = 0; ss < k.n_species; ++ss) {
        const int species = STAGGER ? (int)((ss + blockIdx.x) % (unsigned)k.n_species) : ss;
        const int s_beg = __ldg(k.species_start + species), s_end = __ldg(k.species_start + species + 1);
        const int n_tiles = (s_end - s_beg + TILE - 1) / TILE;
        if (n_tiles == 0) continue;
        if (threadIdx.x == 0) ctl[6 + (ss & 1)] = *reinterpret_cast<volatile int *>(k.tile_counter + species);
        __syncthreads();   // both groups are done with the previous species' tables
        if (ctl[6 + (ss & 1)] >= n_tiles) continue;
        if (TAB_SMEM) {
            const float4 *src = reinterpret_cast<const float4 *>(k.tab.coef + (size_t)species * k.n_species * rows * K_RADIAL);
            const int n4 = k.n_species * rows * (K_RADIAL / 4);
            for (int idx = threadIdx.x; idx < n4; idx += NW * 32)
                *reinterpret_cast<float4 *>(s_tab + (idx >> 3) * TAB_STRIDE_SMEM + 4 * (idx & 7)) = __ldg(src + idx);
            tv.base = s_tab; tv.row_stride = TAB_STRIDE_SMEM; tv.table_stride = rows * TAB_STRIDE_SMEM;
        } else {
            tv.base = k.tab.coef + (size_t)species * k.n_species * rows * K_RADIAL;
            tv.row_stride = K_RADIAL; tv.table_stride = rows * K_RADIAL;
        }
        for (int idx = threadIdx.x; idx < HEAD_L * HEAD_H + HEAD_H + 1; idx += NW * 32)
            hc[idx] = __ldg(k.head_pack + (size_t)species * HP_TOTAL + HP_BIAS + idx);
        if (group == 0) tmem_fill_role(tm_role, k.head_pack + (size_t)species * HP_TOTAL, wg, lane);
        tmem_fence_before_sync();
        __syncthreads();
        tmem_fence_after_sync();

        bool prefetched = false;   // this warp's atom of the coming tile sits in the prefetch buffer
        int look_ahead = -1;       // (group leader) the tile after the current one
        // the group's tiles of this species, claimed one ahead: the first is broadcast here, every later one travels with
        // the barrier between encoding and head
        group_sync(group);
        if (wg == 0 && lane == 0) ctl[2 * group] = atomicAdd(k.tile_counter + species, 1);
        group_sync(group);
        int tile = ctl[2 * group];
        while (tile < n_tiles) {
            if (wg == 0 && lane == 0) look_ahead = atomicAdd(k.tile_counter + species, 1);   // consumed after the encoding
            pc.mark(11);
            const int first = s_beg + tile * TILE;
            const int count = min(TILE, s_end - first);

            // ---------------- Encoding + invariants: warp = atom ----------------
            const bool have = wg < count;
            int i = 0, n_pref = 0, cs = 0;
            double4 pi = make_double4(0.0, 0.0, 0.0, 0.0);
            int64_t beg = 0, end = 0;
            float Pf[4][4];
            int queued = -1;
            float *xrow = sX + wg * X_STRIDE;
            if (have) {
                if (prefetched) {
                    asm volatile("cp.async.wait_group 0;" ::: "memory");
                    __syncwarp();
                    i = pf[PF_IDX];
                    beg = ((int64_t)pf[PF_IDX + 2] << 32) | (unsigned)pf[PF_IDX + 1];
                    end = beg + pf[PF_IDX + 3];
                    n_pref = min(PF_IDX, pf[PF_IDX + 3]);
                    if (L16) cs = lane < 27 ? pf[PF_CS + lane] : 0;
                } else {
                    i = (int)MLIP_CHECK_INDEX(__ldg(k.center_order + first + wg), k.n, k.status);
                    beg = k.nbr_off[i]; end = use_far ? k.nbr_off[i + 1] : beg + k.nbr_near[i];
                    if (L16) cs = cell_base_of_lane(k, i, lane);
                }
                pi = load_pos4(k.pos4 + i);
                n_pairs += encode_atom<TAB_SMEM, L16>(k, tv, pi, beg, end, pq, scr, lane, Pf, queued, pf, n_pref, cs, pc);
                // Eq. 5 (C_l = I): this lane holds rows a = g, g + 8 of channels 8t + j; sum squares over the rows of a block.
                // Rows 1..3 (l = 1) and 4..7 (l = 2) differ in the top bit of g, so one two-step butterfly over the lower
                // bits sums both; l = 2 then takes row 8 (held by g = 0) and the upper half's sum, l = 3 is rows 9..15.
                float part[4][8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float pa = Pf[j & 3][j >> 2], pb = Pf[j & 3][2 + (j >> 2)];
                    float qa = g >= 1 ? pa * pa : 0.f, qb = g >= 1 ? pb * pb : 0.f;
                    qa += __shfl_xor_sync(0xffffffffu, qa, 4);
                    qb += __shfl_xor_sync(0xffffffffu, qb, 4);
                    qa += __shfl_xor_sync(0xffffffffu, qa, 8);
                    qb += __shfl_xor_sync(0xffffffffu, qb, 8);
                    const float upper = __shfl_xor_sync(0xffffffffu, qa, 16);   // g = 0 receives the sum over g = 4..7
                    qb += __shfl_xor_sync(0xffffffffu, qb, 16);
                    part[0][j] = pa;                  // (the values below are those of the storing lanes, g = 0)
                    part[1][j] = qa;
                    part[2][j] = upper + pb * pb;
                    part[3][j] = qb;
                }
                if (g == 0) {
#pragma unroll
                    for (int l = 0; l < 4; ++l) {
                        *reinterpret_cast<float4 *>(xrow + 32 * l + 8 * t) = make_float4(part[l][0], part[l][1], part[l][2], part[l][3]);
                        *reinterpret_cast<float4 *>(xrow + 32 * l + 8 * t + 4) = make_float4(part[l][4], part[l][5], part[l][6], part[l][7]);
                    }
                }
            } else {   // empty slot of a ragged tile: feed zeros to the head
                for (int c = lane; c < N_INV; c += 32) xrow[c] = 0.f;
            }
            if (wg == 0 && lane == 0) ctl[2 * group + 1] = look_ahead;
            pc.mark(7);
            group_sync(group);
            pc.mark(8);
            const int tile_next = ctl[2 * group + 1];

            // ---------------- Regression (and the prefetch for the next tile) ----------------
            NextAtom nx;
            nx.k = &k; nx.sidx = pf; nx.meta = pf + PF_IDX;
            nx.slot = (tile_next < n_tiles && s_beg + tile_next * TILE + wg < s_end) ? s_beg + tile_next * TILE + wg : -1;
            nx.i = 0; nx.beg = 0; nx.end = 0; nx.use_far = use_far; nx.cid = 0;
            head_tile<DET, L16>(k, sX, hb, hc, tm_role, count, first, group, wg, lane, e_sum, nx, pc);
            prefetched = nx.slot >= 0;
            pc.mark(9);

            // ---------------- Derivation ----------------
            if (have) {
                // W_i = dE_i/dP_i (Eq. 7), already in B-fragment order
                const int la = g == 0 ? 0 : (g <= 3 ? 1 : 2), lb = g == 0 ? 2 : 3;
                float da[8], db[8];
                {
                    const float4 a0 = *reinterpret_cast<const float4 *>(xrow + 32 * la + 8 * t), a1 = *reinterpret_cast<const float4 *>(xrow + 32 * la + 8 * t + 4);
                    const float4 b0 = *reinterpret_cast<const float4 *>(xrow + 32 * lb + 8 * t), b1 = *reinterpret_cast<const float4 *>(xrow + 32 * lb + 8 * t + 4);
                    da[0] = a0.x; da[1] = a0.y; da[2] = a0.z; da[3] = a0.w; da[4] = a1.x; da[5] = a1.y; da[6] = a1.z; da[7] = a1.w;
                    db[0] = b0.x; db[1] = b0.y; db[2] = b0.z; db[3] = b0.w; db[4] = b1.x; db[5] = b1.y; db[6] = b1.z; db[7] = b1.w;
                }
                uint32_t Wh[4][4], Wl[4][4];
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const float w0 = g == 0 ? da[ks] : 2.f * da[ks] * Pf[ks][0];          // row a = g,     channel 8t + ks
                    const float w1 = g == 0 ? da[4 + ks] : 2.f * da[4 + ks] * Pf[ks][1];  // row a = g,     channel 8t + 4 + ks
                    const float w2 = 2.f * db[ks] * Pf[ks][2];                            // row a = g + 8, channel 8t + ks
                    const float w3 = 2.f * db[4 + ks] * Pf[ks][3];                        // row a = g + 8, channel 8t + 4 + ks
                    split2_rn(w0, w1, Wh[ks][0], Wh[ks][1], Wl[ks][0], Wl[ks][1]);   // once per atom: the rounded split
                    split2_rn(w2, w3, Wh[ks][2], Wh[ks][3], Wl[ks][2], Wl[ks][3]);
                }
                derive_atom<TAB_SMEM, DET, L16>(k, tv, i, pq, scr, queued, lane, Wh, Wl, vir, pc);
                if (DET) {   // fold this atom's virial in now: lane sums in a fixed order, then integers
#pragma unroll
                    for (int q = 0; q < 9; ++q) {
                        float x = vir[q];
#pragma unroll
                        for (int o = 16; o; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
                        if (lane == q) vir_fx += rint((double)x * VIRIAL_FX);
                        vir[q] = 0.f;
                    }
                }
            }
            pc.mark(10);
            tile = tile_next;
        }
    }
    pc.flush(k.acc, lane);

    // per-warp totals -> global accumulators
    if (DET) {
        if (lane < 9) atomicAdd(reinterpret_cast<unsigned long long *>(k.acc_fx + 1 + lane), (unsigned long long)(long long)vir_fx);
        if (lane == 0) atomicAdd(reinterpret_cast<unsigned long long *>(k.acc_fx), (unsigned long long)(long long)e_sum);
    } else {
#pragma unroll
        for (int q = 0; q < 9; ++q) {
            float x = vir[q];
#pragma unroll
            for (int o = 16; o; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
            if (lane == 0) atomicAdd(&k.acc[ACC_VIRIAL + q], (double)x);
        }
        if (lane == 0) atomicAdd(&k.acc[ACC_ENERGY], e_sum);
    }
    if (lane == 0) atomicAdd(k.pair_counter, n_pairs);
    tmem_fence_before_sync();
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tm_base), "r"(TM_COLS) : "memory");
}

// ---------------- host side ----------------
int table_smem_words(const mlip_ctx *c) { return c->cfg.n_species * (c->cfg.table_knots + 3) * TAB_STRIDE_SMEM; }
bool tables_fit_smem(const mlip_ctx *c) { return FIXED_WORDS + table_smem_words(c) <= SMEM_LIMIT_WORDS; }

int upload_head(mlip_ctx *c, const double *w) {
    const int C = c->cfg.n_species;
    float *host = (float *)calloc((size_t)C * HP_TOTAL, sizeof(float));
    if (!host) return MLIP_ERR_OOM;
    for (int s = 0; s < C; ++s) {
        const double *src = w + (size_t)s * HEAD_NET;
        float *hp = host + (size_t)s * HP_TOTAL;
        float *fwd = hp + HP_FWD, *bwd = hp + HP_BWD;
        int in = N_INV;
        for (int L = 0; L < HEAD_L; ++L) {
            const int nks = in / 8;
            // forward: A[m][k] = W[m][k]; record (mt, ks), lane (g, t):
            //   a0 = W[16mt+g][8ks+t], a1 = W[16mt+g+8][8ks+t], a2 = W[16mt+g][8ks+t+4], a3 = W[16mt+g+8][8ks+t+4]
            for (int mt = 0; mt < 4; ++mt)
                for (int ks = 0; ks < nks; ++ks)
                    for (int lane = 0; lane < 32; ++lane) {
                        const int g = lane >> 2, t = lane & 3;
                        float *rec = fwd + ((size_t)(mt * nks + ks) * 32 + lane) * 4;
                        rec[0] = (float)src[(16 * mt + g) * in + 8 * ks + t];
                        rec[1] = (float)src[(16 * mt + g + 8) * in + 8 * ks + t];
                        rec[2] = (float)src[(16 * mt + g) * in + 8 * ks + t + 4];
                        rec[3] = (float)src[(16 * mt + g + 8) * in + 8 * ks + t + 4];
                    }
            // reverse: A[m][k] = W[k][m] (m = input, k = neuron); record (mt, ks)
            for (int mt = 0; mt < in / 16; ++mt)
                for (int ks = 0; ks < 8; ++ks)
                    for (int lane = 0; lane < 32; ++lane) {
                        const int g = lane >> 2, t = lane & 3;
                        float *rec = bwd + ((size_t)(mt * 8 + ks) * 32 + lane) * 4;
                        rec[0] = (float)src[(8 * ks + t) * in + 16 * mt + g];
                        rec[1] = (float)src[(8 * ks + t) * in + 16 * mt + g + 8];
                        rec[2] = (float)src[(8 * ks + t + 4) * in + 16 * mt + g];
                        rec[3] = (float)src[(8 * ks + t + 4) * in + 16 * mt + g + 8];
                    }
            for (int o = 0; o < HEAD_H; ++o) hp[HP_BIAS + L * HEAD_H + o] = (float)src[in * HEAD_H + o];
            src += in * HEAD_H + HEAD_H;
            fwd += (size_t)4 * nks * 128;
            bwd += (size_t)(in / 16) * 8 * 128;
            in = HEAD_H;
        }
        for (int o = 0; o < HEAD_H + 1; ++o) hp[HP_WOUT + o] = (float)src[o];
    }
    cudaError_t e = cudaMalloc(&c->head_w, sizeof(float) * (size_t)C * HP_TOTAL);
    if (e == cudaSuccess) e = cudaMemcpy(c->head_w, host, sizeof(float) * (size_t)C * HP_TOTAL, cudaMemcpyHostToDevice);
    free(host);
    if (e != cudaSuccess) { c->err = cudaGetErrorString(e); return MLIP_ERR_CUDA; }
    c->resident += sizeof(float) * (size_t)C * HP_TOTAL;
    return MLIP_OK;
}

// Deterministic mode: integer sums -> the float / double outputs the rest of the library reads.
__global__ void k_fixed_finish(int64_t n, const long long *__restrict__ force_fx, const long long *__restrict__ acc_fx,
                               float4 *__restrict__ force, double *__restrict__ acc) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) {
        const double inv = 1.0 / (double)FORCE_FX;
        force[i] = make_float4((float)((double)force_fx[3 * i] * inv), (float)((double)force_fx[3 * i + 1] * inv),
                               (float)((double)force_fx[3 * i + 2] * inv), 0.f);
    }
    if (i == 0) {
        acc[ACC_ENERGY] = (double)acc_fx[0] / ENERGY_FX;
        for (int q = 0; q < 9; ++q) acc[ACC_VIRIAL + q] = (double)acc_fx[1 + q] / VIRIAL_FX;
    }
}

int launch_megakernel(mlip_ctx *c, cudaStream_t s) {
    const int64_t n = c->n;
    const bool det = c->cfg.force_mode == 1;
    if (det) MLIP_CUDA_TRY(c, cudaMemsetAsync(c->force_fx, 0, sizeof(long long) * 3 * n, s));
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->force, 0, sizeof(float4) * n, s));
    MLIP_CUDA_TRY(c, cudaMemsetAsync(c->launch_block, 0, LAUNCH_CLEAR_BYTES, s));   // tile and pair counters, integer and fp64 accumulators
    const int64_t tiles_max = (n + TILE - 1) / TILE + c->cfg.n_species;
    const int blocks = (int)std::min<int64_t>(tiles_max, (int64_t)c->n_sm);
    const bool in_smem = tables_fit_smem(c);
    const int tab_words = in_smem ? table_smem_words(c) : 0;
    const size_t smem_bytes = sizeof(float) * (size_t)(FIXED_WORDS + tab_words);
    // instantiations: tables in shared / global memory x floating-point / integer scatter x int32 / 16-bit lists, and the
    // shared-memory ones again with staggered species for small systems
    using Kernel = void (*)(KernelArgs, int);
    static const Kernel kernels[12] = {k_mega<false, false, false, false>, k_mega<false, false, true, false>, k_mega<false, true, false, false>,
                                       k_mega<false, true, true, false>,   k_mega<true, false, false, false>, k_mega<true, false, true, false>,
                                       k_mega<true, true, false, false>,   k_mega<true, true, true, false>,   k_mega<true, false, false, true>,
                                       k_mega<true, false, true, true>,    k_mega<true, true, false, true>,   k_mega<true, true, true, true>};
    const bool stagger = in_smem && n < STAGGER_BELOW_ATOMS;
    if (!c->kernel_ready) {
        for (int q = 0; q < 12; ++q) {
            const size_t bytes = sizeof(float) * (size_t)(FIXED_WORDS + (q >= 4 ? tab_words : 0));
            cudaError_t e = cudaFuncSetAttribute((const void *)kernels[q], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
            if (e != cudaSuccess) { c->err = std::string("fused kernel shared memory: ") + cudaGetErrorString(e); return MLIP_ERR_CUDA; }
        }
        c->kernel_ready = true;
    }
    KernelArgs k;
    k.n = n; k.n_species = c->cfg.n_species; k.grid = c->grid; k.rc2 = c->cfg.r_cut * c->cfg.r_cut; k.tab = c->tab;
    k.pos4 = c->pos4; k.center_order = c->center_order; k.species_start = c->species_start;
    k.nbr_off = c->nbr_off; k.nbr_near = c->nbr_near; k.far_flag = c->far_flag; k.nbr = c->nbr; k.nbr16 = reinterpret_cast<const uint16_t *>(c->nbr); k.cell_id = c->cell_id; k.cell_start = c->cell_start;
    k.nbr_cap = c->nbr_cap; k.head_pack = c->head_w; k.force = c->force; k.e_atom = c->e_atom;
    k.force_fx = c->force_fx; k.acc_fx = c->acc_fx;
    k.acc = c->acc; k.pair_counter = c->pair_counter; k.status = c->status; k.tile_counter = c->tile_counter;
    const int slot = (int)(c->ev_count % mlip_ctx::EV_POOL);
    MLIP_CUDA_TRY(c, cudaEventRecord(c->ev[2 * slot], s));
    kernels[(stagger ? 8 : in_smem ? 4 : 0) + (det ? 2 : 0) + (c->list16 ? 1 : 0)]<<<blocks, NW * 32, smem_bytes, s>>>(k, tab_words);
    if (det) {
        k_fixed_finish<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(n, c->force_fx, c->acc_fx, c->force, c->acc);
        c->launches += 1;
    }
    MLIP_CUDA_TRY(c, cudaEventRecord(c->ev[2 * slot + 1], s));
    c->ev_count += 1;
    c->launches += 1;
    MLIP_CUDA_TRY(c, cudaGetLastError());
    return MLIP_OK;
}

}  // namespace mlip
