// Stage (b) in ONE pass for bf16 weights and the half-density patterns (2:4, 4:8): Eq. 4 / Eq. 5 score, N:M
// selection, and every output of the selection -- mask bits, pruned copy, compressed values and metadata -- from a
// single read of W (Section 3, "Extension to N:M Sparsity": mask and compressed form come from the same selection).
// Per weight: 2 bytes read, 2 + 1 + 0.125 + 0.125 written; the two-pass route (dass_score_nm, then
// dass_compress_nm) moves 7.375 bytes for the same result.
//
// Data movement: a warp unit is 8 rows x 256 columns (4 KB).  Units arrive through TMA (cp.async.bulk.tensor, one
// box per unit, issued by one lane) into a per-warp ring of shared-memory slots guarded by mbarriers, so the next
// unit is in flight while the current one is worked on, no lane computes a load address, and everything outside the
// matrix reads as zero.  A lane then owns 8 consecutive columns (one 16-byte vector per row); stores are 16-byte and
// coalesced (a warp row is one contiguous 512-byte segment).
//
// The selection is arranged so that most of its work leaves the integer / logic pipe (the busy one):
//   * p = fl32(|w| * scale); rounding is monotone, so an order between rounded products is an order between the
//     exact ones.  The cut value t of a group (its n_keep-th largest p) comes from a short min / max cascade
//     (6 operations for 2 of 4 with a three-input max, 25 for 4 of 8).
//   * d = p - t has its sign bit set exactly when p < t.  One byte permute with sign replication turns the two
//     differences of a word's two bf16 into that word's "pruned" lane mask (0xffff per pruned element), which
//     serves the pruned copy (one AND-NOT per word) and, for 2:4 row groups, the compaction itself: the first
//     survivor of a column is row 0, else row 1, else row 2, a two-level select on lane masks (2 logic ops per
//     output word).
//   * keep bytes (bit j = column j) are picked out of the lane masks with constant masks; four rows' bytes are
//     transposed across a quad of lanes with two shuffles so that each lane stores one whole 32-bit mask word.
//   * a group holds a tie across the cut exactly when more than n_keep of its products are >= t: one population
//     count per four keep bytes.  Only then is the order not proven and the group redone with exact double
//     products (rare on real data, always correct).
// Every mbarrier wait is bounded; a wait that runs out records DASS_ERR_TIMEOUT in a status word of the library
// (read by dass_prune_status) and the warp returns.
#include "tc_common.cuh"

namespace dass {

struct PruneParams {
    const uint16_t *W;
    uint16_t *Wp;        // nullable
    uint32_t *mask;      // nullable
    uint16_t *values;    // nullable (then meta is null too)
    uint32_t *meta;
    const float *norm;
    int64_t rows, cols, ld;
    int64_t wpr;         // mask words per row
    int64_t vcols;       // elements per row of the values matrix
    int64_t mwpl;        // metadata words per line
    int64_t strips, blocks;          // 256-column strips, 8-row blocks
    int64_t fast;        // units along the direction a warp walks (the scales stay the same along it)
    int runs;            // a line of `fast` units is cut into this many near-equal runs, one per warp
    int ctas_per_line;   // per-column scales: CTAs that share one strip (runs / warps per CTA, rounded up)
    int scale_mode;
    float alpha;
    int vec_ok;          // value rows start 16-byte (row groups) / 8-byte (column groups) aligned
    uint32_t box_bytes;  // bytes of one TMA box (box columns x box rows x 2)
    uint32_t pitch16;    // row pitch of a box in shared memory, in 16-byte vectors
};

namespace {

constexpr int PN_THREADS = 128;
constexpr int PN_MIN_BLOCKS = 4;     // 16 warps per SM at up to 128 registers
constexpr int PN_COLS = 256;
constexpr int PN_ROWS = 8;

// Out of line: the double-precision sqrt / pow sequences run once per strip or per 32 rows only.
__device__ __noinline__ float pn_scale_of(float n, int mode, float alpha) { return scale_from_norm(n, mode, alpha); }

__device__ __forceinline__ uint32_t pn_prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

__device__ __forceinline__ float max3f(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

__device__ __forceinline__ uint32_t wsel(const uint4 &v, int k) { return k == 0 ? v.x : k == 1 ? v.y : k == 2 ? v.z : v.w; }
__device__ __forceinline__ uint32_t &wref(uint4 &v, int k) { return k == 0 ? v.x : k == 1 ? v.y : k == 2 ? v.z : v.w; }

// fl32(|low bf16 of word| * s) and the same for the high one.  The low half is moved up with a multiply so that it
// runs beside the float pipe rather than on the logic pipe.
__device__ __forceinline__ float prod_lo(uint32_t word, float s) { return fabsf(__uint_as_float(word * 65536u)) * s; }
__device__ __forceinline__ float prod_hi(uint32_t word, float s) { return fabsf(__uint_as_float(word & 0xffff0000u)) * s; }

// Second largest of four.
__device__ __forceinline__ float cut_2of4(float a, float b, float c, float d)
{
    const float h1 = fmaxf(a, b), l1 = fminf(a, b), h2 = fmaxf(c, d), l2 = fminf(c, d);
    return max3f(fminf(h1, h2), l1, l2);
}

__device__ __forceinline__ void sort4_desc(float &a, float &b, float &c, float &d)
{
    const float h1 = fmaxf(a, b), l1 = fminf(a, b), h2 = fmaxf(c, d), l2 = fminf(c, d);
    const float m = fminf(h1, h2), l = fmaxf(l1, l2);
    a = fmaxf(h1, h2);
    b = fmaxf(m, l);
    c = fminf(m, l);
    d = fminf(l1, l2);
}

// Fourth largest of eight: both halves sorted, then the merge rule "the k-th largest of two sorted lists is the
// largest of min(a_i, b_(k-2-i)) and of a_(k-1), b_(k-1)".
__device__ __forceinline__ float cut_4of8(const float (&x)[8])
{
    float a0 = x[0], a1 = x[1], a2 = x[2], a3 = x[3], b0 = x[4], b1 = x[5], b2 = x[6], b3 = x[7];
    sort4_desc(a0, a1, a2, a3);
    sort4_desc(b0, b1, b2, b3);
    return max3f(max3f(a3, b3, fminf(a0, b2)), fminf(a1, b1), fminf(a2, b0));
}

template <int M>
__device__ __forceinline__ float cut_of(const float (&x)[M])
{
    if constexpr (M == 4) return cut_2of4(x[0], x[1], x[2], x[3]);
    else return cut_4of8(x);
}

// Lane mask of a word from the differences of its two elements: 0xffff where the difference is negative.
__device__ __forceinline__ uint32_t pruned_lanes(float d_lo, float d_hi)
{
    return pn_prmt(__float_as_uint(d_lo), __float_as_uint(d_hi), 0xFFBBu);
}

// Bytes (bit j = column j) of the lane-mask words of two rows, in the low 16 bits of the result (row a in byte 0,
// row b in byte 1).  Even columns sit in the low lanes and land on their bit directly; odd columns sit in the high
// lanes, are picked 16 bits up and folded down at the end.
__device__ __forceinline__ uint32_t bytes_of_lanes2(const uint32_t (&za)[4], const uint32_t (&zb)[4])
{
    uint32_t x = za[0] & 0x00020001u;
    x |= za[1] & 0x00080004u;
    x |= za[2] & 0x00200010u;
    x |= za[3] & 0x00800040u;
    x |= zb[0] & 0x02000100u;
    x |= zb[1] & 0x08000400u;
    x |= zb[2] & 0x20001000u;
    x |= zb[3] & 0x80004000u;
    return x | (x >> 16);
}

// "Pruned" bytes of four rows in one word (byte i = row i).
__device__ __forceinline__ uint32_t bytes_of_lanes4(const uint32_t (&z0)[4], const uint32_t (&z1)[4], const uint32_t (&z2)[4],
                                                    const uint32_t (&z3)[4])
{
    return pn_prmt(bytes_of_lanes2(z0, z1), bytes_of_lanes2(z2, z3), 0x5410u);
}

// 16-bit lane masks (0xffff per set bit) of an 8-bit byte: bit j -> sign of byte j, then sign-replicating permutes.
__device__ __forceinline__ void lanes_of_byte(uint32_t byte, uint32_t (&m)[4])
{
    const uint32_t zlo = (byte & 0xfu) * 0x10204080u;
    const uint32_t zhi = ((byte >> 4) & 0xfu) * 0x10204080u;
    m[0] = pn_prmt(zlo, 0u, 0x9988u);
    m[1] = pn_prmt(zlo, 0u, 0xbbaau);
    m[2] = pn_prmt(zhi, 0u, 0x9988u);
    m[3] = pn_prmt(zhi, 0u, 0xbbaau);
}

// 4 x 4 byte transpose across a quad of lanes: on entry byte i of x belongs to row i (this lane's 8 columns); on
// return lane k of the quad holds the word of row k (byte l from lane l of the quad).  Whole warp must call.
__device__ __forceinline__ uint32_t quad_transpose(uint32_t x, uint32_t sel1, uint32_t sel2)
{
    const uint32_t y = __shfl_xor_sync(FULL_MASK, x, 1);
    const uint32_t z = pn_prmt(x, y, sel1);
    const uint32_t y2 = __shfl_xor_sync(FULL_MASK, z, 2);
    return pn_prmt(z, y2, sel2);
}

// Stores the first n of a lane's 8 elements; one 16-byte store when all 8 exist and the address is known to be aligned.
__device__ __forceinline__ void store_row8(uint16_t *dst, const uint4 &v, int n, bool vec = true)
{
    if (vec && n == 8) {
        DASS_ST_CS(reinterpret_cast<uint4 *>(dst), v);
    } else {
        for (int j = 0; j < n; ++j) {
            const uint32_t w = wsel(v, j >> 1);
            DASS_ST(&dst[j], (uint16_t)((j & 1) ? (w >> 16) : (w & 0xffffu)));
        }
    }
}

// ---------------------------------------------------------------- exact selection (rare path)
template <int R> struct Tile { uint4 v[R]; };
template <int R> struct KeepBytes { uint32_t k[R]; };
struct Scale8 { float s[8]; };

// Row groups: M rows x 8 columns, scales per column (norm_cols) or per row; keep byte per row.
template <int M>
__device__ __noinline__ KeepBytes<M> exact_rows(Tile<M> t, Scale8 sc, int norm_cols)
{
    KeepBytes<M> out;
#pragma unroll
    for (int q = 0; q < M; ++q) out.k[q] = 0u;
    for (int j = 0; j < 8; ++j) {
        double s[M];
#pragma unroll
        for (int q = 0; q < M; ++q) {
            const uint32_t w = wsel(t.v[q], j >> 1);
            const uint32_t fb = (j & 1) ? (w & 0x7fff0000u) : ((w & 0x7fffu) << 16);
            s[q] = (double)__uint_as_float(fb) * (double)(norm_cols ? sc.s[j] : sc.s[q]);
        }
        const uint32_t kg = select_group<M>(s, M / 2);
#pragma unroll
        for (int q = 0; q < M; ++q) out.k[q] |= ((kg >> q) & 1u) << j;
    }
    return out;
}

// Column groups: 4 rows x 8 columns (8 / M groups per row); keep byte per row.
template <int M>
__device__ __noinline__ KeepBytes<4> exact_cols(Tile<4> t, Scale8 sc, int norm_cols)
{
    KeepBytes<4> out;
    for (int i = 0; i < 4; ++i) {
        uint32_t keep = 0u;
#pragma unroll
        for (int g = 0; g < 8 / M; ++g) {
            double s[M];
#pragma unroll
            for (int q = 0; q < M; ++q) {
                const int j = g * M + q;
                const uint32_t w = wsel(t.v[i], j >> 1);
                const uint32_t fb = (j & 1) ? (w & 0x7fff0000u) : ((w & 0x7fffu) << 16);
                s[q] = (double)__uint_as_float(fb) * (double)(norm_cols ? sc.s[j] : sc.s[i]);
            }
            keep |= select_group<M>(s, M / 2) << (g * M);
        }
        out.k[i] = keep;
    }
    return out;
}

// bit j of a byte -> bit 4j
__device__ __forceinline__ uint32_t spread_bits(uint32_t b)
{
    uint32_t x = (b | (b << 12)) & 0x000F000Fu;
    x = (x | (x << 6)) & 0x03030303u;
    return (x | (x << 3)) & 0x11111111u;
}

// nibble made of bit j of each of the four bytes of x (byte a -> bit a)
__device__ __forceinline__ uint32_t gather_bit4(uint32_t x, int j) { return (((x >> j) & 0x01010101u) * 0x10204080u) >> 28; }

// ---------------------------------------------------------------- work decomposition
// A unit is 8 rows x 256 columns.  A warp walks a run of consecutive units in the direction along which its
// scales stay the same: down a strip when the scales belong to columns, across the strips of one 8-row block when
// they belong to rows.  A line of units along that direction is cut into p.runs near-equal runs.  CTAs are small
// (4 warps, a few units per warp) and numerous, so the hardware's block scheduler evens out the SMs.
//   per-column scales: the warps of a CTA take consecutive runs of ONE strip and share its 256 scales through
//                      shared memory;
//   per-row scales:    the warps of a CTA take the same strip range at consecutive row blocks.
constexpr int PN_STAGES = 3;
constexpr uint32_t PN_SLOT_BYTES = PN_ROWS * PN_COLS * 2;           // 4 KB: one full box
constexpr uint32_t PN_WARPS = PN_THREADS / 32;
constexpr uint32_t PN_SMEM_BYTES = PN_WARPS * PN_STAGES * PN_SLOT_BYTES + PN_WARPS * PN_STAGES * 8 + 128;
constexpr unsigned long long PN_WAIT_NS = 2000000000ull;            // a wait gives up after 2 s

__device__ int g_prune_status = 0;     // DASS_OK or DASS_ERR_TIMEOUT; read and cleared through dass_prune_status

template <bool NORM_COLS>
struct Run {
    int line;        // the fixed index: strip (per-column scales) or row block (per-row scales)
    int f0, f1;      // units [f0, f1) along the walking direction; empty for a warp without work
    __device__ __forceinline__ void set(const PruneParams &p, int warp_in_cta)
    {
        int r;
        bool live;
        if constexpr (NORM_COLS) {
            line = (int)(blockIdx.x / (unsigned)p.ctas_per_line);
            r = (int)(blockIdx.x % (unsigned)p.ctas_per_line) * (int)PN_WARPS + warp_in_cta;
            live = r < p.runs;
        } else {
            line = (int)(blockIdx.x / (unsigned)p.runs) * (int)PN_WARPS + warp_in_cta;
            r = (int)(blockIdx.x % (unsigned)p.runs);
            live = line < p.blocks;
        }
        f0 = live ? (int)((int64_t)r * p.fast / p.runs) : 0;
        f1 = live ? (int)((int64_t)(r + 1) * p.fast / p.runs) : 0;
    }
    __device__ __forceinline__ int strip(int f) const { return NORM_COLS ? line : f; }
    __device__ __forceinline__ int blk(int f) const { return NORM_COLS ? f : line; }
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y) : "memory");
}

// Bounded wait of the whole warp on one of its slots.  False after PN_WAIT_NS.
__device__ __forceinline__ bool slot_wait(uint32_t bar, uint32_t parity)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t spin = 1; spin < (1u << 30); ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 63u) == 0 && global_ns() - t0 > PN_WAIT_NS) return false;
    }
    return false;
}

// The TMA-fed ring of a warp: PN_STAGES slots of one box each, one mbarrier per slot.
template <bool NORM_COLS>
struct UnitRing {
    uint32_t slots, bars;            // shared-memory addresses of this warp's slots and barriers
    const uint8_t *generic;          // generic pointer to slot 0
    int f_pre;                       // next unit of the run to fetch
    int slot = 0;
    uint32_t phase = 0;

    __device__ __forceinline__ void issue(const CUtensorMap *map, const PruneParams &p, const Run<NORM_COLS> &run, int into, int lane)
    {
        if (lane == 0 && f_pre < run.f1) {
            const uint32_t bar = bars + 8u * into;
            mbar_arrive_expect_tx(bar, p.box_bytes);
            tma_load_2d(slots + into * PN_SLOT_BYTES, map, bar, run.strip(f_pre) * PN_COLS, run.blk(f_pre) * PN_ROWS);
        }
        ++f_pre;
    }
    __device__ __forceinline__ void start(uint8_t *smem_aligned, int warp_in_cta, const CUtensorMap *map, const PruneParams &p,
                                          const Run<NORM_COLS> &run, int lane)
    {
        generic = smem_aligned + warp_in_cta * PN_STAGES * PN_SLOT_BYTES;
        slots = smem_u32(generic);
        bars = smem_u32(smem_aligned + PN_WARPS * PN_STAGES * PN_SLOT_BYTES) + warp_in_cta * PN_STAGES * 8;
        if (lane == 0) {
#pragma unroll
            for (int s = 0; s < PN_STAGES; ++s) mbar_init(bars + 8u * s, 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
        f_pre = run.f0;
#pragma unroll
        for (int s = 0; s < PN_STAGES - 1; ++s) issue(map, p, run, s, lane);
    }
    // Refills the slot consumed one iteration ago, then waits for the current unit.  Returns its tile (16-byte
    // vectors, row pitch p.pitch16) or nullptr when the wait ran out.
    __device__ __forceinline__ const uint4 *next(const CUtensorMap *map, const PruneParams &p, const Run<NORM_COLS> &run, int lane)
    {
        __syncwarp();                  // every lane is done reading the slot that is refilled now
        issue(map, p, run, slot == 0 ? PN_STAGES - 1 : slot - 1, lane);
        const bool ok = slot_wait(bars + 8u * slot, phase);
        const uint4 *tile = reinterpret_cast<const uint4 *>(generic + slot * PN_SLOT_BYTES);
        if (++slot == PN_STAGES) { slot = 0; phase ^= 1u; }
        return ok ? tile : nullptr;
    }
    // After a failed wait: record it and give the copies still in flight one more bounded chance to land.
    __device__ __forceinline__ void fail(int lane)
    {
        if (lane == 0) atomicExch(&g_prune_status, (int)DASS_ERR_TIMEOUT);
#pragma unroll
        for (int s = 0; s < PN_STAGES; ++s) {
            slot_wait(bars + 8u * s, 0u);
            slot_wait(bars + 8u * s, 1u);
        }
    }
};

// Scales of a run.  Per-column: the CTA evaluates its strip's 256 scales once (two per thread) into shared memory
// and a lane picks up its 8.  Per-row: lanes 0..7 evaluate the block's 8 rows and the warp shares them.
// Every thread of the CTA must call this (it holds a barrier in the per-column case).
template <bool NORM_COLS>
__device__ __forceinline__ void run_scales(const PruneParams &p, const Run<NORM_COLS> &run, float *cta_scales, int lane, float (&s)[8])
{
    if constexpr (NORM_COLS) {
        for (int e = threadIdx.x; e < PN_COLS; e += PN_THREADS) {
            const int64_t c = (int64_t)run.line * PN_COLS + e;
            cta_scales[e] = c < p.cols ? pn_scale_of(DASS_LD(&p.norm[c]), p.scale_mode, p.alpha) : 0.0f;
        }
        __syncthreads();
        const float4 a = reinterpret_cast<const float4 *>(cta_scales)[lane * 2];
        const float4 b = reinterpret_cast<const float4 *>(cta_scales)[lane * 2 + 1];
        s[0] = a.x; s[1] = a.y; s[2] = a.z; s[3] = a.w; s[4] = b.x; s[5] = b.y; s[6] = b.z; s[7] = b.w;
    } else {
        const int64_t r = (int64_t)run.line * PN_ROWS + (lane & 7);
        const float mine = (run.f1 > run.f0 && r < p.rows) ? pn_scale_of(DASS_LD(&p.norm[r]), p.scale_mode, p.alpha) : 0.0f;
#pragma unroll
        for (int q = 0; q < 8; ++q) s[q] = __shfl_sync(FULL_MASK, mine, q);
    }
}

// ---------------------------------------------------------------- one unit, groups along the rows (gate / up)
// ALL: every output is wanted (compile-time, no tests of the output pointers).  FULL: the unit lies inside the
// matrix and every store is a whole aligned vector (no edge handling at all).
template <int M, bool NORM_COLS, bool ALL, bool FULL>
__device__ __forceinline__ void rows_unit(const PruneParams &p, const uint4 *tile, const float (&sc)[8], const uint32_t *spread_lut,
                                          int64_t r0, int64_t c0, int lane, uint32_t sel1, uint32_t sel2)
{
    constexpr int G = PN_ROWS / M;          // row groups per unit
    constexpr int K = M / 2;                // survivors per group
    const bool want_mask = ALL || p.mask != nullptr, want_pruned = ALL || p.Wp != nullptr, want_values = ALL || p.values != nullptr;
    const int64_t left = p.cols - c0;
    const int nvalid = FULL ? 8 : (left >= 8 ? 8 : (left > 0 ? (int)left : 0));
    const uint32_t valid = (1u << nvalid) - 1u;
    const uint32_t valid4 = valid * 0x01010101u;
    const bool quad_live = FULL || (c0 & ~(int64_t)31) < p.cols;      // the quad's 32 columns hold at least one column
    const uint32_t pitch = FULL ? 32u : p.pitch16;
    uint16_t *const wp = p.Wp + r0 * p.ld + c0;
    uint16_t *const vp = p.values + (r0 / M) * K * p.vcols + c0;
    uint32_t *const kp = p.mask + (r0 + (lane & 3)) * p.wpr + (c0 >> 5);

#pragma unroll
    for (int g = 0; g < G; ++g) {
        if (!FULL && r0 + g * M >= p.rows) break;          // warp-uniform; rows is a multiple of M: a group is whole or absent
        uint4 v[M];
#pragma unroll
        for (int q = 0; q < M; ++q) v[q] = tile[(g * M + q) * pitch + lane];
        // ---- selection: pruned-lane masks of the group's M rows
        uint32_t Z[M][4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float pe[M], po[M];
#pragma unroll
            for (int q = 0; q < M; ++q) {
                const uint32_t w = wsel(v[q], k);
                pe[q] = prod_lo(w, NORM_COLS ? sc[2 * k] : sc[g * M + q]);
                po[q] = prod_hi(w, NORM_COLS ? sc[2 * k + 1] : sc[g * M + q]);
            }
            const float te = cut_of<M>(pe), to = cut_of<M>(po);
#pragma unroll
            for (int q = 0; q < M; ++q) Z[q][k] = pruned_lanes(__fsub_rn(pe[q], te), __fsub_rn(po[q], to));
        }
        uint32_t keep[M / 4];              // byte i of keep[h] = keep byte of row 4h + i
        uint32_t count = 0u;
#pragma unroll
        for (int h = 0; h < M / 4; ++h) {
            keep[h] = ~bytes_of_lanes4(Z[4 * h], Z[4 * h + 1], Z[4 * h + 2], Z[4 * h + 3]);
            if (!FULL) keep[h] &= valid4;
            count += __popc(keep[h]);
        }
        if (count != (uint32_t)(K * nvalid)) {
            // more than n_keep products at or above the cut somewhere: a tie across the cut -> exact products
            Tile<M> t;
            Scale8 s8;
#pragma unroll
            for (int q = 0; q < M; ++q) t.v[q] = v[q];
#pragma unroll
            for (int j = 0; j < 8; ++j) s8.s[j] = NORM_COLS ? sc[j] : (j < M ? sc[g * M + (j < M ? j : 0)] : 0.0f);
            const KeepBytes<M> e = exact_rows<M>(t, s8, NORM_COLS ? 1 : 0);
#pragma unroll
            for (int h = 0; h < M / 4; ++h)
                keep[h] = ((e.k[4 * h] & valid) | ((e.k[4 * h + 1] & valid) << 8) | ((e.k[4 * h + 2] & valid) << 16) |
                           ((e.k[4 * h + 3] & valid) << 24));
#pragma unroll
            for (int q = 0; q < M; ++q) {
                uint32_t m[4];
                lanes_of_byte(e.k[q], m);
#pragma unroll
                for (int k = 0; k < 4; ++k) Z[q][k] = ~m[k];
            }
        }

        // ---- mask words: lane k of a quad stores the word of row 4h + k
        if (want_mask) {
#pragma unroll
            for (int h = 0; h < M / 4; ++h) {
                const uint32_t word = quad_transpose(keep[h], sel1, sel2);
                if (quad_live) DASS_ST(&kp[(g * M + 4 * h) * p.wpr], word);
            }
        }
        if (!FULL && nvalid == 0) continue;        // no shuffles below: lanes are independent from here on

        // ---- survivors in place (pruned -> +0)
        uint4 P[M == 4 ? 4 : 1];          // 2:4 compacts from the pruned rows; 4:8 only stores them
#pragma unroll
        for (int q = 0; q < M; ++q) {
            uint4 &row = P[M == 4 ? q : 0];
#pragma unroll
            for (int k = 0; k < 4; ++k) wref(row, k) = wsel(v[q], k) & ~Z[q][k];
            if (want_pruned) {
                if (FULL) DASS_ST_CS(reinterpret_cast<uint4 *>(wp + (g * M + q) * p.ld), row);
                else store_row8(wp + (g * M + q) * p.ld, row, nvalid);
            }
        }
        if (!want_values) continue;

        // ---- compressed values + metadata
        const int64_t line = r0 / M + g;
        uint16_t *const vg = vp + g * K * p.vcols;
        if constexpr (M == 4) {
            // first survivor of a column: row 0, else row 1, else row 2; second: row 3, else row 2, else row 1
            uint4 o0, o1;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                wref(o0, k) = wsel(P[0], k) | (Z[0][k] & (wsel(P[1], k) | (Z[1][k] & wsel(P[2], k))));
                wref(o1, k) = wsel(P[3], k) | (Z[3][k] & (wsel(P[2], k) | (Z[2][k] & wsel(P[1], k))));
            }
            if (FULL) {
                DASS_ST_CS(reinterpret_cast<uint4 *>(vg), o0);
                DASS_ST_CS(reinterpret_cast<uint4 *>(vg + p.vcols), o1);
            } else {
                store_row8(vg, o0, nvalid, p.vec_ok != 0);
                store_row8(vg + p.vcols, o1, nvalid, p.vec_ok != 0);
            }
            // nibble of column j = pos_lo | pos_hi << 2; as bytes over the 8 columns:
            //   pos_lo bit 0 = ~K0 & K1, bit 1 = ~K0 & ~K1, pos_hi bit 0 = K3 | ~K2, bit 1 = K3 | K2
            const uint32_t k0 = keep[0], k1 = keep[0] >> 8, k2 = keep[0] >> 16, k3 = keep[0] >> 24;
            const uint32_t b0 = (~k0 & k1) & 0xffu, b1 = ~(k0 | k1) & 0xffu, b2 = (k3 | ~k2) & 0xffu, b3 = (k3 | k2) & 0xffu;
            uint32_t fields = spread_lut[b0] | (spread_lut[b1] << 1) | (spread_lut[b2] << 2) | (spread_lut[b3] << 3);
            if (!FULL) fields &= spread_lut[valid] * 15u;
            DASS_ST(&p.meta[line * p.mwpl + (c0 >> 3)], fields);
        } else {
            // Row q of the group goes to output row k = number of kept rows above it (bit-sliced over the 8
            // columns); for every possible (q, k) the byte "kept and count == k" becomes lane masks.
            uint4 o[K];
#pragma unroll
            for (int k = 0; k < K; ++k) o[k] = make_uint4(0u, 0u, 0u, 0u);
            uint32_t cnt0 = 0u, cnt1 = 0u;     // bit-sliced count (a kept row has at most K - 1 = 3 kept rows above it)
#pragma unroll
            for (int q = 0; q < M; ++q) {
                const uint32_t m = (keep[q >> 2] >> (8 * (q & 3))) & 0xffu;
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    if (k <= q && q - k <= M - K) {
                        const uint32_t e = ((k & 1) ? cnt0 : ~cnt0) & ((k & 2) ? cnt1 : ~cnt1) & m;
                        uint32_t lm[4];
                        lanes_of_byte(e, lm);
#pragma unroll
                        for (int w = 0; w < 4; ++w) wref(o[k], w) |= wsel(v[q], w) & lm[w];
                    }
                }
                const uint32_t carry = cnt0 & m;
                cnt0 ^= m;
                cnt1 ^= carry;
            }
#pragma unroll
            for (int k = 0; k < K; ++k) {
                if (FULL) DASS_ST_CS(reinterpret_cast<uint4 *>(vg + k * p.vcols), o[k]);
                else store_row8(vg + k * p.vcols, o[k], nvalid, p.vec_ok != 0);
            }
            // field of column j = its 8-bit keep mask (bit q = row q): the bit transpose of the keep bytes
            uint32_t f_lo = 0u, f_hi = 0u;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t colmask = gather_bit4(keep[0], j) | (gather_bit4(keep[M / 4 - 1], j) << 4);
                if (j < 4) f_lo |= colmask << (8 * j);
                else f_hi |= colmask << (8 * (j - 4));
            }
            DASS_ST(&p.meta[line * p.mwpl + (c0 >> 2)], f_lo);
            if (FULL || nvalid > 4) DASS_ST(&p.meta[line * p.mwpl + (c0 >> 2) + 1], f_hi);
        }
    }
}

}  // namespace

template <int M, bool NORM_COLS, bool ALL>
__global__ void __launch_bounds__(PN_THREADS, PN_MIN_BLOCKS) prune_rows_bf16_kernel(const __grid_constant__ CUtensorMap map_w, const PruneParams p)
{
    extern __shared__ uint8_t pn_smem_raw[];
    __shared__ uint32_t spread_lut[256];    // bit j of a byte -> bit 4j (2:4 metadata: bytes of position bits -> nibbles)
    __shared__ __align__(16) float cta_scales[NORM_COLS ? PN_COLS : 4];
    if constexpr (M == 4)
        for (int e = threadIdx.x; e < 256; e += PN_THREADS) spread_lut[e] = spread_bits(e);
    uint8_t *smem = pn_smem_raw + ((128u - (smem_u32(pn_smem_raw) & 127u)) & 127u);
    const int lane = threadIdx.x & 31;
    const uint32_t sel1 = (lane & 1) ? 0x3715u : 0x6240u;
    const uint32_t sel2 = (lane & 2) ? 0x3276u : 0x5410u;
    Run<NORM_COLS> run;
    run.set(p, threadIdx.x >> 5);
    float sc[8];
    run_scales<NORM_COLS>(p, run, cta_scales, lane, sc);
    if constexpr (M == 4 && !NORM_COLS) __syncthreads();      // the look-up table (per-column scales: run_scales held the barrier)
    UnitRing<NORM_COLS> ring;
    ring.start(smem, threadIdx.x >> 5, &map_w, p, run, lane);

    for (int f = run.f0; f < run.f1; ++f) {
        const uint4 *tile = ring.next(&map_w, p, run, lane);
        if (tile == nullptr) { ring.fail(lane); return; }
        const int strip = run.strip(f);
        const int64_t r0 = (int64_t)run.blk(f) * PN_ROWS;
        const int64_t c0 = (int64_t)strip * PN_COLS + lane * 8;
        // whole unit inside the matrix and every store a whole aligned vector: the branch-free path (warp-uniform)
        const bool full = ((int64_t)strip + 1) * PN_COLS <= p.cols && r0 + PN_ROWS <= p.rows && p.vec_ok != 0;
        if (full) rows_unit<M, NORM_COLS, ALL, true>(p, tile, sc, spread_lut, r0, c0, lane, sel1, sel2);
        else rows_unit<M, NORM_COLS, ALL, false>(p, tile, sc, spread_lut, r0, c0, lane, sel1, sel2);
    }
}

namespace {

// ---------------------------------------------------------------- groups along the columns (down)
// Shared-memory table indexed by a row's keep byte: the permute selectors that compact the survivors and, for 2:4,
// the metadata byte.
//   M = 4: x = selector of group 0 | selector of group 1 << 16 (each picks two bf16 out of a word pair),
//          y = metadata byte (two nibbles pos_lo | pos_hi << 2)
//   M = 8: x, y = selectors of output words 0 and 1: low 16 bits pick a 16-bit half out of each word pair,
//          high 16 bits pick between the two results
__device__ __forceinline__ uint2 cols_table_entry(uint32_t byte, int m)
{
    if (m == 4) {
        uint32_t sel = 0u, meta = 0u;
        for (int g = 0; g < 2; ++g) {
            const uint32_t nib = (byte >> (4 * g)) & 0xfu;
            const uint32_t lo = nib ? (uint32_t)(__ffs(nib) - 1) : 0u;
            const uint32_t hi = nib ? (uint32_t)(31 - __clz(nib)) : 0u;
            sel |= (0x1010u + 0x22u * lo + 0x2200u * hi) << (16 * g);
            meta |= (lo | (hi << 2)) << (4 * g);
        }
        return make_uint2(sel, meta);
    }
    uint32_t s[2] = {0u, 0u};
    uint32_t rest = byte;
    for (int w = 0; w < 2; ++w) {
        const uint32_t pa = rest ? (uint32_t)(__ffs(rest) - 1) : 0u;
        rest &= rest - 1u;
        const uint32_t pb = rest ? (uint32_t)(__ffs(rest) - 1) : 0u;
        rest &= rest - 1u;
        const uint32_t i = 2u * (pa & 3u), j = 2u * (pb & 3u);
        const uint32_t s1 = (i | ((i + 1u) << 4)) | ((j | ((j + 1u) << 4)) << 8);
        const uint32_t s2 = 0x3210u + (pa >> 2) * 0x0044u + (pb >> 2) * 0x4400u;
        s[w] = s1 | (s2 << 16);
    }
    return make_uint2(s[0], s[1]);
}

template <int M, bool NORM_COLS, bool ALL, bool FULL>
__device__ __forceinline__ void cols_unit(const PruneParams &p, const uint4 *tile, const float (&sc)[8], const uint2 *table,
                                          int64_t r0, int64_t c0, int lane, uint32_t sel1, uint32_t sel2)
{
    constexpr int G = 8 / M;                 // groups inside a lane's 8 columns
    const bool want_mask = ALL || p.mask != nullptr, want_pruned = ALL || p.Wp != nullptr, want_values = ALL || p.values != nullptr;
    const int64_t left = p.cols - c0;
    const int nvalid = FULL ? 8 : (left >= 8 ? 8 : (left > 0 ? (int)left : 0));     // a multiple of M
    const int nout = nvalid / 2;
    const uint32_t valid = (1u << nvalid) - 1u;
    const bool quad_live = FULL || (c0 & ~(int64_t)31) < p.cols;
    const uint32_t pitch = FULL ? 32u : p.pitch16;
    uint16_t *const wp = p.Wp + r0 * p.ld + c0;
    uint16_t *const vp = p.values + r0 * p.vcols + (c0 >> 1);
    uint32_t *const kp = p.mask + (r0 + (lane & 3)) * p.wpr + (c0 >> 5);
    uint32_t *const mp = p.meta + (r0 + (lane & 3)) * p.mwpl + (c0 >> 5);

#pragma unroll
    for (int h = 0; h < PN_ROWS / 4; ++h) {
        const int64_t rh = r0 + 4 * h;
        if (!FULL && rh >= p.rows) break;           // warp-uniform
        const int nrows = FULL ? 4 : (p.rows - rh >= 4 ? 4 : (int)(p.rows - rh));
        uint4 v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = tile[(4 * h + i) * pitch + lane];
        uint32_t Z[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float pr[8];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t w = wsel(v[i], k);
                pr[2 * k] = prod_lo(w, NORM_COLS ? sc[2 * k] : sc[4 * h + i]);
                pr[2 * k + 1] = prod_hi(w, NORM_COLS ? sc[2 * k + 1] : sc[4 * h + i]);
            }
            float t[G];
            if constexpr (M == 4) {
                t[0] = cut_2of4(pr[0], pr[1], pr[2], pr[3]);
                t[1] = cut_2of4(pr[4], pr[5], pr[6], pr[7]);
            } else {
                t[0] = cut_4of8(pr);
            }
#pragma unroll
            for (int k = 0; k < 4; ++k)
                Z[i][k] = pruned_lanes(__fsub_rn(pr[2 * k], t[(2 * k) / M]), __fsub_rn(pr[2 * k + 1], t[(2 * k + 1) / M]));
        }
        const uint32_t rows4 = nrows == 4 ? 0xffffffffu : ((1u << (8 * nrows)) - 1u);
        const uint32_t valid4 = (valid * 0x01010101u) & rows4;
        uint32_t keep = ~bytes_of_lanes4(Z[0], Z[1], Z[2], Z[3]);
        if (!FULL) keep &= valid4;
        if (__popc(keep) * 2 != (FULL ? 32 : __popc(valid4))) {
            // more than n_keep products at or above some group's cut: a tie across the cut -> exact products
            Tile<4> t;
            Scale8 s8;
#pragma unroll
            for (int i = 0; i < 4; ++i) t.v[i] = v[i];
#pragma unroll
            for (int j = 0; j < 8; ++j) s8.s[j] = NORM_COLS ? sc[j] : (j < 4 ? sc[4 * h + (j < 4 ? j : 0)] : 0.0f);
            const KeepBytes<4> e = exact_cols<M>(t, s8, NORM_COLS ? 1 : 0);
            keep = (e.k[0] | (e.k[1] << 8) | (e.k[2] << 16) | (e.k[3] << 24)) & valid4;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t m[4];
                lanes_of_byte(e.k[i], m);
#pragma unroll
                for (int k = 0; k < 4; ++k) Z[i][k] = ~m[k];
            }
        }
        const bool row_live = FULL || (lane & 3) < nrows;
        if (want_mask) {
            const uint32_t word = quad_transpose(keep, sel1, sel2);
            if (quad_live && row_live) DASS_ST(&kp[4 * h * p.wpr], word);
        }
        uint32_t metab = 0u;               // byte i = metadata byte of row i
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (FULL || (i < nrows && nvalid > 0)) {      // lanes past the last column only skip stores
                if (want_pruned) {
                    uint4 P;
#pragma unroll
                    for (int k = 0; k < 4; ++k) wref(P, k) = wsel(v[i], k) & ~Z[i][k];
                    if (FULL) DASS_ST_CS(reinterpret_cast<uint4 *>(wp + (4 * h + i) * p.ld), P);
                    else store_row8(wp + (4 * h + i) * p.ld, P, nvalid);
                }
                if (want_values) {
                    const uint32_t kb = (keep >> (8 * i)) & 0xffu;
                    const uint2 e = table[kb];
                    uint32_t o0, o1;
                    if constexpr (M == 4) {
                        o0 = pn_prmt(v[i].x, v[i].y, e.x);
                        o1 = pn_prmt(v[i].z, v[i].w, e.x >> 16);
                        metab |= e.y << (8 * i);
                    } else {
                        o0 = pn_prmt(pn_prmt(v[i].x, v[i].y, e.x), pn_prmt(v[i].z, v[i].w, e.x), e.x >> 16);
                        o1 = pn_prmt(pn_prmt(v[i].x, v[i].y, e.y), pn_prmt(v[i].z, v[i].w, e.y), e.y >> 16);
                    }
                    uint16_t *dst = vp + (4 * h + i) * p.vcols;
                    if (FULL || (nout == 4 && p.vec_ok)) {
                        DASS_ST_CS(reinterpret_cast<uint2 *>(dst), make_uint2(o0, o1));
                    } else {
                        for (int k = 0; k < nout; ++k) {
                            const uint32_t ow = k < 2 ? o0 : o1;
                            DASS_ST(&dst[k], (uint16_t)((k & 1) ? (ow >> 16) : (ow & 0xffffu)));
                        }
                    }
                }
            }
        }
        if (want_values) {
            // 2:4: nibbles pos_lo | pos_hi << 2; 4:8: the 8-bit keep mask of the group, i.e. the keep byte
            const uint32_t word = quad_transpose(M == 4 ? metab : keep, sel1, sel2);
            if (quad_live && row_live) DASS_ST(&mp[4 * h * p.mwpl], word);
        }
    }
}

}  // namespace

template <int M, bool NORM_COLS, bool ALL>
__global__ void __launch_bounds__(PN_THREADS, PN_MIN_BLOCKS) prune_cols_bf16_kernel(const __grid_constant__ CUtensorMap map_w, const PruneParams p)
{
    extern __shared__ uint8_t pn_smem_raw[];
    __shared__ uint2 table[256];
    __shared__ __align__(16) float cta_scales[NORM_COLS ? PN_COLS : 4];
    for (int e = threadIdx.x; e < 256; e += PN_THREADS) table[e] = cols_table_entry(e, M);
    uint8_t *smem = pn_smem_raw + ((128u - (smem_u32(pn_smem_raw) & 127u)) & 127u);
    const int lane = threadIdx.x & 31;
    const uint32_t sel1 = (lane & 1) ? 0x3715u : 0x6240u;
    const uint32_t sel2 = (lane & 2) ? 0x3276u : 0x5410u;
    Run<NORM_COLS> run;
    run.set(p, threadIdx.x >> 5);
    float sc[8];
    run_scales<NORM_COLS>(p, run, cta_scales, lane, sc);
    if constexpr (!NORM_COLS) __syncthreads();                // the table (per-column scales: run_scales held the barrier)
    UnitRing<NORM_COLS> ring;
    ring.start(smem, threadIdx.x >> 5, &map_w, p, run, lane);

    for (int f = run.f0; f < run.f1; ++f) {
        const uint4 *tile = ring.next(&map_w, p, run, lane);
        if (tile == nullptr) { ring.fail(lane); return; }
        const int strip = run.strip(f);
        const int64_t r0 = (int64_t)run.blk(f) * PN_ROWS;
        const int64_t c0 = (int64_t)strip * PN_COLS + lane * 8;
        const bool full = ((int64_t)strip + 1) * PN_COLS <= p.cols && r0 + PN_ROWS <= p.rows && p.vec_ok != 0;
        if (full) cols_unit<M, NORM_COLS, ALL, true>(p, tile, sc, table, r0, c0, lane, sel1, sel2);
        else cols_unit<M, NORM_COLS, ALL, false>(p, tile, sc, table, r0, c0, lane, sel1, sel2);
    }
}

int device_sm_count();   // dass_abi.cu
bool tile_map_bf16(CUtensorMap *map, const void *ptr, int64_t rows, int64_t cols, int64_t ld, int box_cols, int box_rows);   // calib_tc.cu

template <typename Kernel>
static cudaError_t launch_prune(Kernel kernel, DeviceMask &configured, const CUtensorMap &map, const PruneParams &p,
                                int64_t grid, cudaStream_t st)
{
    const cudaError_t e = ensure_dynamic_smem(kernel, (int)PN_SMEM_BYTES, configured);
    if (e != cudaSuccess) return e;
    kernel<<<(unsigned)grid, PN_THREADS, PN_SMEM_BYTES, st>>>(map, p);
    return cudaGetLastError();
}

template <int M, bool NORM_COLS, bool ALL>
static cudaError_t launch_axis(bool group_cols, const CUtensorMap &map, const PruneParams &p, int64_t grid, cudaStream_t st)
{
    static DeviceMask cfg_rows{0ull}, cfg_cols{0ull};                // per device, per instantiation
    return group_cols ? launch_prune(prune_cols_bf16_kernel<M, NORM_COLS, ALL>, cfg_cols, map, p, grid, st)
                      : launch_prune(prune_rows_bf16_kernel<M, NORM_COLS, ALL>, cfg_rows, map, p, grid, st);
}

// Fused stage (b) for bf16 weights and n_keep = m / 2, m in {4, 8}; arguments validated by the caller.
cudaError_t prune_nm_bf16_launch(const void *W, int64_t rows, int64_t cols, int64_t ld,
                                 const float *norm, bool norm_cols, float alpha, int m, bool group_cols,
                                 uint32_t *mask_bits, void *W_pruned, void *values, uint32_t *meta, cudaStream_t st)
{
    PruneParams p;
    p.W = static_cast<const uint16_t *>(W);
    p.Wp = static_cast<uint16_t *>(W_pruned);
    p.mask = mask_bits;
    p.values = static_cast<uint16_t *>(values);
    p.meta = meta;
    p.norm = norm;
    p.rows = rows; p.cols = cols; p.ld = ld;
    p.wpr = (cols + 31) / 32;
    const bool two_four = m == 4;
    if (group_cols) {
        p.vcols = cols / 2;
        p.mwpl = (cols + 31) / 32;          // 4 bits per 4 columns or 8 bits per 8 columns: one bit per column
        p.vec_ok = (cols % 8 == 0) && ((reinterpret_cast<uintptr_t>(values) & 7u) == 0);
    } else {
        p.vcols = cols;
        const int fpw = two_four ? 8 : 4;
        p.mwpl = (cols + fpw - 1) / fpw;
        p.vec_ok = (cols % 8 == 0) && ((reinterpret_cast<uintptr_t>(values) & 15u) == 0);
    }
    p.strips = (cols + PN_COLS - 1) / PN_COLS;
    p.blocks = (rows + PN_ROWS - 1) / PN_ROWS;
    p.scale_mode = (int)scale_mode_for(alpha);
    p.alpha = alpha;
    if (rows > 0x7fffffffll - PN_ROWS || cols > 0x7fffffffll - PN_COLS) return cudaErrorInvalidValue;
    // one TMA box per unit; a box never exceeds the matrix (narrow or short matrices get a smaller box)
    const int box_cols = cols >= PN_COLS ? PN_COLS : (int)((cols + 7) / 8 * 8);
    const int box_rows = rows >= PN_ROWS ? PN_ROWS : (int)rows;
    p.box_bytes = (uint32_t)(box_cols * box_rows * 2);
    p.pitch16 = (uint32_t)(box_cols / 8);
    CUtensorMap map;
    if (!tile_map_bf16(&map, W, rows, cols, ld, box_cols, box_rows)) return cudaErrorInvalidValue;

    // Runs: about 8 CTAs per resident slot so that the block scheduler can even out the SMs, but at least 4 units
    // per warp so that a warp's start-up (scales, first tile) stays small beside its work.
    p.fast = norm_cols ? p.blocks : p.strips;
    const int64_t lines = norm_cols ? p.strips : p.blocks;
    const int64_t units = p.fast * lines;
    const int64_t target_ctas = (int64_t)device_sm_count() * PN_MIN_BLOCKS * 8;
    int64_t per_warp = units / (target_ctas * PN_WARPS);
    per_warp = per_warp < 4 ? 4 : (per_warp > 64 ? 64 : per_warp);
    int64_t runs = (p.fast + per_warp - 1) / per_warp;
    if (runs > 0x7fffffffll) return cudaErrorInvalidValue;
    p.runs = (int)runs;
    p.ctas_per_line = (int)((runs + PN_WARPS - 1) / PN_WARPS);
    const int64_t grid = norm_cols ? lines * p.ctas_per_line : ((lines + PN_WARPS - 1) / PN_WARPS) * runs;
    if (grid > 0x7fffffffll) return cudaErrorInvalidValue;

    const bool all = mask_bits && W_pruned && values;
    if (m == 4) {
        if (norm_cols) return all ? launch_axis<4, true, true>(group_cols, map, p, grid, st) : launch_axis<4, true, false>(group_cols, map, p, grid, st);
        return all ? launch_axis<4, false, true>(group_cols, map, p, grid, st) : launch_axis<4, false, false>(group_cols, map, p, grid, st);
    }
    if (norm_cols) return all ? launch_axis<8, true, true>(group_cols, map, p, grid, st) : launch_axis<8, true, false>(group_cols, map, p, grid, st);
    return all ? launch_axis<8, false, true>(group_cols, map, p, grid, st) : launch_axis<8, false, false>(group_cols, map, p, grid, st);
}

// Reads and clears the status word of the one-pass kernels (waits for the stream).
cudaError_t prune_status_read(int *host_value, cudaStream_t st)
{
    cudaError_t e = cudaMemcpyFromSymbolAsync(host_value, g_prune_status, sizeof(int), 0, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return e;
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return e;
    if (*host_value != 0) {
        const int zero = 0;
        e = cudaMemcpyToSymbolAsync(g_prune_status, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    }
    return e;
}

}  // namespace dass
