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
#include "stream_units.cuh"

namespace dass {

struct PruneParams : UnitGrid {
    const uint16_t *W;
    uint16_t *Wp;        // nullable
    uint32_t *mask;      // nullable
    uint16_t *values;    // nullable (then meta is null too)
    uint32_t *meta;
    const float *norm;
    int64_t ld;
    int64_t wpr;         // mask words per row
    int64_t vcols;       // elements per row of the values matrix
    int64_t mwpl;        // metadata words per line
    int scale_mode;
    float alpha;
    int vec_ok;          // value rows start 16-byte (row groups) / 8-byte (column groups) aligned
};

namespace {

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
        if (tile == nullptr) { ring.fail(lane, p.status); return; }
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
        if (tile == nullptr) { ring.fail(lane, p.status); return; }
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

__device__ int g_stage_b_status = 0;     // DASS_OK or DASS_ERR_TIMEOUT; read and cleared through dass_prune_status

// Device address of the status word of the TMA-fed stage-(b) kernels (looked up once per device).
int *stage_b_status_word()
{
    static std::atomic<int *> cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    int *ptr = cached[dev].load(std::memory_order_acquire);
    if (!ptr) {
        void *sym = nullptr;
        if (cudaGetSymbolAddress(&sym, g_stage_b_status) != cudaSuccess) return nullptr;
        ptr = static_cast<int *>(sym);
        cached[dev].store(ptr, std::memory_order_release);
    }
    return ptr;
}

// Fills the decomposition of a [rows x cols] bf16 matrix into units and runs, encodes its tensor map and returns the
// grid size.  Runs: about 8 CTAs per resident slot so that the block scheduler can even out the SMs, but at least 4
// units per warp so that a warp's start-up (scales, first tile) stays small beside its work.
cudaError_t unit_grid_setup(UnitGrid &g, CUtensorMap *map, int64_t *grid, const void *W, int64_t rows, int64_t cols, int64_t ld,
                            bool walk_down)
{
    if (rows > 0x7fffffffll - PN_ROWS || cols > 0x7fffffffll - PN_COLS) return cudaErrorInvalidValue;
    g.rows = rows; g.cols = cols;
    g.strips = (cols + PN_COLS - 1) / PN_COLS;
    g.blocks = (rows + PN_ROWS - 1) / PN_ROWS;
    // one TMA box per unit; a box never exceeds the matrix (narrow or short matrices get a smaller box)
    const int box_cols = cols >= PN_COLS ? PN_COLS : (int)((cols + 7) / 8 * 8);
    const int box_rows = rows >= PN_ROWS ? PN_ROWS : (int)rows;
    g.box_bytes = (uint32_t)(box_cols * box_rows * 2);
    g.pitch16 = (uint32_t)(box_cols / 8);
    if (!tile_map_bf16(map, W, rows, cols, ld, box_cols, box_rows)) return cudaErrorInvalidValue;
    g.fast = walk_down ? g.blocks : g.strips;
    const int64_t lines = walk_down ? g.strips : g.blocks;
    const int64_t units = g.fast * lines;
    const int64_t target_ctas = (int64_t)device_sm_count() * PN_MIN_BLOCKS * 8;
    int64_t per_warp = units / (target_ctas * PN_WARPS);
    per_warp = per_warp < 4 ? 4 : (per_warp > 64 ? 64 : per_warp);
    const int64_t runs = (g.fast + per_warp - 1) / per_warp;
    if (runs > 0x7fffffffll) return cudaErrorInvalidValue;
    g.runs = (int)runs;
    g.ctas_per_line = (int)((runs + PN_WARPS - 1) / PN_WARPS);
    *grid = walk_down ? lines * g.ctas_per_line : ((lines + PN_WARPS - 1) / PN_WARPS) * runs;
    if (*grid > 0x7fffffffll) return cudaErrorInvalidValue;
    g.status = stage_b_status_word();
    return cudaSuccess;
}

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
    p.ld = ld;
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
    p.scale_mode = (int)scale_mode_for(alpha);
    p.alpha = alpha;
    CUtensorMap map;
    int64_t grid = 0;
    const cudaError_t ge = unit_grid_setup(p, &map, &grid, W, rows, cols, ld, norm_cols);
    if (ge != cudaSuccess) return ge;

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
    cudaError_t e = cudaMemcpyFromSymbolAsync(host_value, g_stage_b_status, sizeof(int), 0, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return e;
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return e;
    if (*host_value != 0) {
        const int zero = 0;
        e = cudaMemcpyToSymbolAsync(g_stage_b_status, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    }
    return e;
}

}  // namespace dass
