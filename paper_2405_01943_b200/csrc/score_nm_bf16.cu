// Stage (b) for bf16 weights: Eq. 4 / Eq. 5 score and N:M selection (mask and pruned copy), tuned to stay under the
// HBM roofline.  The patterns with n_keep = m / 2 (2:4, 4:8) are served by the one-pass kernels of prune_nm_bf16.cu;
// these kernels serve the other bf16 patterns (1:4, 3:4, 1:8 ... 7:8).
//
// Same tiling as the generic kernels in score_nm.cu (a lane owns 8 consecutive columns = one 16-byte
// vector; a warp row is one contiguous 512-byte segment), but the selection is done with 32-bit
// integer and bit-sliced logic instead of per-element double arithmetic:
//
//   * p = fl32(|w| * scale).  Rounding is monotone, so p_b > p_a proves score_b > score_a for the exact
//     products.  A group's products are sorted with a min / max network, which gives the cut value t (the
//     n_keep-th largest) and the value below it; every element is then compared with t by the sign of the float
//     difference p - t (never wrong), shifted into a bit-sliced word with one funnel shift (bit j of a word =
//     column j of the lane's tile).
//   * only when the two values at the cut are EQUAL is the order not proven; the lane then recomputes its
//     tile's keep bits with exact double products (rare on real data, always correct).
//   * pruned weights: keep bits are spread to byte sign bits with one multiply and expanded to 16-bit
//     masks with the sign-replicating byte permute.
//
// Work is split in units of one 8-row (column groups) or M-row (row groups) slab of 256 columns; a warp
// takes a contiguous range of units that walks down a 256-column strip, so per-column scales are
// evaluated once per strip and per-row scales once per 32 rows.
#include "dass_device.cuh"

namespace dass {

struct ScoreFastParams {
    const uint16_t *W;
    uint16_t *Wp;        // nullable
    uint32_t *mask;      // nullable
    const float *norm;
    int64_t rows, cols, ld;
    int64_t wpr;         // mask words per row
    int64_t units_per_strip, units;
    int n_keep;
    int scale_mode;
    float alpha;
};

constexpr int F_THREADS = 256;
constexpr int F_MIN_BLOCKS = 4;      // CTAs per SM the 2:4 row-group kernel is compiled for (64 registers: measured best)
constexpr int F_COLS = 256;          // columns per warp strip
// prefetch depth of the shared-memory slab ring (slabs of R rows x 512 bytes per warp)
__host__ __device__ constexpr int ring_stages(int rows_per_unit) { return rows_per_unit >= 8 ? 2 : 3; }
__host__ __device__ constexpr int ring_bytes(int rows_per_unit) { return (F_THREADS / 32) * ring_stages(rows_per_unit) * rows_per_unit * 512; }
constexpr int F_SLAB = 4;            // rows per unit when groups run along the columns

// Out of line on purpose: the double-precision sqrt / pow sequences would otherwise inflate the register
// budget of the streaming loops, and they run once per strip or per 32 rows only.
__device__ __noinline__ float scale_of(float n, int mode, float alpha) { return scale_from_norm(n, mode, alpha); }

// 16-byte asynchronous copy global -> shared (src_bytes = 0 writes zeros and reads nothing)
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc, int src_bytes)
{
    if (src_bytes != 0 && !DASS_ACCESS_OK(gsrc, 16)) src_bytes = 0;     // checking build: an outside source reads as zeros
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;"
                 ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Prefetch ring of a warp: STAGES slabs of R rows x 32 lanes x 16 bytes in shared memory.  A lane only ever
// reads back the 16 bytes it copied itself, so the per-thread wait_group is the only synchronisation needed.
template <int R, int STAGES>
struct SlabRing {
    uint4 *buf;   // this warp's [STAGES][R][32]
    __device__ __forceinline__ uint4 *slot(int stage, int row, int lane) const { return buf + (stage * R + row) * 32 + lane; }
    // starts the copy of the unit at `cur` (rows r0..r0+R-1 of the lane's 8 columns) into `stage` and
    // commits the group; `live` is false past the warp's last unit (an empty group keeps the count uniform)
    __device__ __forceinline__ void issue(const ScoreFastParams &p, int strip, int g, bool live, int stage, int lane) const
    {
        if (live) {
            const int64_t r0 = (int64_t)g * R;
            const int64_t c0 = (int64_t)strip * F_COLS + lane * 8;
            const bool col_ok = c0 < p.cols;
            const uint16_t *src = p.W + r0 * p.ld + c0;
#pragma unroll
            for (int i = 0; i < R; ++i) {
                const bool ok = col_ok && (r0 + i < p.rows);
                cp_async16(slot(stage, i, lane), ok ? (const void *)src : (const void *)p.W, ok ? 16 : 0);
                src += p.ld;
            }
        }
        cp_async_commit();
    }
};

// Position of a unit: which 256-column strip and which slab inside it.  Units of a warp are consecutive,
// so the position is advanced instead of being divided out of the unit index each time.
struct UnitCursor {
    int strip, g;
    __device__ __forceinline__ void advance(int units_per_strip)
    {
        if (++g == units_per_strip) { g = 0; ++strip; }
    }
};

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// fl32(|element| * scale); element = low (hi == false) or high half of a word of two bf16.  The low half is
// moved up with a multiply so that it runs on the FMA pipe (the integer/logic pipe is the busy one here).
__device__ __forceinline__ float prod_of(uint32_t word, bool hi, float scale)
{
    const uint32_t fb = hi ? (word & 0xffff0000u) : (word * 65536u);
    return fabsf(__uint_as_float(fb)) * scale;
}

// Selection inside a group of M rounded products: the products are sorted with a small min / max network (5
// comparators for M = 4, 19 for M = 8) and every element is compared with the n_keep-th largest, t.  "p >= t" is
// the keep rule whenever t is strictly above the next value: monotone rounding then proves the same for the exact
// products, and equal products on one side of the cut need no order.  threshold_group shifts "p_q < t" (the sign
// of p_q - t, which floating-point subtraction never gets wrong) into the bit-sliced words D and returns true if
// the two values at the cut are equal (order not proven: the lane then takes the exact path).
__device__ __forceinline__ void cmp_exchange(float &hi, float &lo)
{
    const float a = fmaxf(hi, lo), b = fminf(hi, lo);
    hi = a;
    lo = b;
}

// The n_keep-th and (n_keep+1)-th largest of M rounded products (M = 4: 5-comparator network, M = 8: 19).
template <int M>
__device__ __forceinline__ void cut_values(const float (&pf)[M], int n_keep, float &t, float &next)
{
    float s[M];
#pragma unroll
    for (int q = 0; q < M; ++q) s[q] = pf[q];
    if constexpr (M == 4) {
        cmp_exchange(s[0], s[1]); cmp_exchange(s[2], s[3]);
        cmp_exchange(s[0], s[2]); cmp_exchange(s[1], s[3]);
        cmp_exchange(s[1], s[2]);                         // s[0] >= s[1] >= s[2] >= s[3]
        switch (n_keep) {                                 // n_keep in 1..3, the same for every lane
        case 1: t = s[0]; next = s[1]; break;
        case 2: t = s[1]; next = s[2]; break;
        default: t = s[2]; next = s[3]; break;
        }
    } else {
        cmp_exchange(s[0], s[1]); cmp_exchange(s[2], s[3]); cmp_exchange(s[4], s[5]); cmp_exchange(s[6], s[7]);
        cmp_exchange(s[0], s[2]); cmp_exchange(s[1], s[3]); cmp_exchange(s[4], s[6]); cmp_exchange(s[5], s[7]);
        cmp_exchange(s[1], s[2]); cmp_exchange(s[5], s[6]); cmp_exchange(s[0], s[4]); cmp_exchange(s[3], s[7]);
        cmp_exchange(s[1], s[5]); cmp_exchange(s[2], s[6]);
        cmp_exchange(s[1], s[4]); cmp_exchange(s[3], s[6]);
        cmp_exchange(s[2], s[4]); cmp_exchange(s[3], s[5]);
        cmp_exchange(s[3], s[4]);                         // s[0] >= s[1] >= ... >= s[7]
        switch (n_keep) {                                 // n_keep in 1..7, the same for every lane
        case 1: t = s[0]; next = s[1]; break;
        case 2: t = s[1]; next = s[2]; break;
        case 3: t = s[2]; next = s[3]; break;
        case 4: t = s[3]; next = s[4]; break;
        case 5: t = s[4]; next = s[5]; break;
        case 6: t = s[5]; next = s[6]; break;
        default: t = s[6]; next = s[7]; break;
        }
    }
}

template <int M>
__device__ __forceinline__ bool threshold_group(const float (&pf)[M], int n_keep, uint32_t (&D)[M])
{
    float t, next;
    cut_values<M>(pf, n_keep, t, next);
#pragma unroll
    for (int q = 0; q < M; ++q) D[q] = __funnelshift_l(__float_as_uint(__fsub_rn(pf[q], t)), D[q], 1);
    return t == next;
}

// 16-bit lane masks for the 8 bf16 of a chunk from an 8-bit keep byte, applied in place.
__device__ __forceinline__ void apply_keep_byte(uint4 &v, uint32_t keep)
{
    const uint32_t zlo = (keep & 0xfu) * 0x10204080u;    // bit j -> sign bit of byte j
    const uint32_t zhi = ((keep >> 4) & 0xfu) * 0x10204080u;
    v.x &= prmt(zlo, 0u, 0x9988u);
    v.y &= prmt(zlo, 0u, 0xbbaau);
    v.z &= prmt(zhi, 0u, 0x9988u);
    v.w &= prmt(zhi, 0u, 0xbbaau);
}

__device__ __forceinline__ uint32_t word_of(const uint4 &v, int k) { return k == 0 ? v.x : k == 1 ? v.y : k == 2 ? v.z : v.w; }

__device__ __forceinline__ void store_chunk(uint16_t *dst, const uint4 &v, int nvalid)
{
    if (nvalid == 8) {
        DASS_ST_CS(reinterpret_cast<uint4 *>(dst), v);
    } else {
        for (int j = 0; j < nvalid; ++j) {
            const uint32_t w = word_of(v, j >> 1);
            DASS_ST(&dst[j], (uint16_t)((j & 1) ? (w >> 16) : (w & 0xffffu)));
        }
    }
}

// ---------------------------------------------------------------- exact fallback (rare)
template <int R> struct TileWords { uint4 v[R]; };
template <int R> struct KeepWords { uint32_t k[R]; };
struct Scales8 { float s[8]; };

// Row groups: tile = M rows x 8 columns; returns for each row its 8-bit keep byte (bit j = column j).
template <int M>
__device__ __noinline__ KeepWords<M> exact_keep_rows(TileWords<M> t, Scales8 sc /* per column or per row */,
                                                     int norm_cols, int n_keep)
{
    KeepWords<M> out;
#pragma unroll
    for (int q = 0; q < M; ++q) out.k[q] = 0u;
    for (int j = 0; j < 8; ++j) {
        double s[M];
#pragma unroll
        for (int q = 0; q < M; ++q) {
            const uint32_t w = word_of(t.v[q], j >> 1);
            const uint32_t fb = (j & 1) ? (w & 0x7fff0000u) : ((w & 0x7fffu) << 16);
            s[q] = (double)__uint_as_float(fb) * (double)(norm_cols ? sc.s[j] : sc.s[q]);
        }
        const uint32_t kg = select_group<M>(s, n_keep);
#pragma unroll
        for (int q = 0; q < M; ++q) out.k[q] |= ((kg >> q) & 1u) << j;
    }
    return out;
}

// Column groups: tile = F_SLAB rows x 8 columns; returns for each row its 8-bit keep byte.
template <int M>
__device__ __noinline__ KeepWords<F_SLAB> exact_keep_cols(TileWords<F_SLAB> t, Scales8 sc, int norm_cols, int n_keep)
{
    KeepWords<F_SLAB> out;
    for (int i = 0; i < F_SLAB; ++i) {
        uint32_t keep = 0u;
#pragma unroll
        for (int g = 0; g < 8 / M; ++g) {
            double s[M];
#pragma unroll
            for (int q = 0; q < M; ++q) {
                const int j = g * M + q;
                const uint32_t w = word_of(t.v[i], j >> 1);
                const uint32_t fb = (j & 1) ? (w & 0x7fff0000u) : ((w & 0x7fffu) << 16);
                s[q] = (double)__uint_as_float(fb) * (double)(norm_cols ? sc.s[j] : sc.s[i]);
            }
            keep |= select_group<M>(s, n_keep) << (g * M);
        }
        out.k[i] = keep;
    }
    return out;
}

// ---------------------------------------------------------------- groups along the rows (gate / up)
template <int M, bool NORM_COLS>
__global__ void __launch_bounds__(F_THREADS, M == 8 ? 2 : F_MIN_BLOCKS) score_rows_bf16_kernel(const ScoreFastParams p)
{
    constexpr int STAGES = ring_stages(M);
    extern __shared__ uint4 ring_mem[];
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (F_THREADS / 32) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (F_THREADS / 32);
    const int64_t u_begin = p.units * warp / nwarps;
    const int64_t u_end = p.units * (warp + 1) / nwarps;
    SlabRing<M, STAGES> ring;
    ring.buf = ring_mem + (threadIdx.x >> 5) * (STAGES * M * 32);
    const int ups = (int)p.units_per_strip;
    UnitCursor cur, pre;
    cur.strip = (int)(u_begin / p.units_per_strip);
    cur.g = (int)(u_begin - (int64_t)cur.strip * p.units_per_strip);
    pre = cur;
    int64_t u_pre = u_begin;
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        ring.issue(p, pre.strip, pre.g, u_pre < u_end, s, lane);
        pre.advance(ups);
        ++u_pre;
    }

    int64_t cached_strip = -1, cached_base = -1;
    float sc[8];          // per-column scales of the strip (NORM_COLS)
    float lane_scale = 0.0f;   // scale of row cached_base + lane (!NORM_COLS)
    int nvalid = 0;
    int64_t c0 = 0;
    int stage = 0;

    for (int64_t u = u_begin; u < u_end; ++u, cur.advance(ups)) {
        const int64_t strip = cur.strip;
        const int64_t r0 = (int64_t)cur.g * M;
        if (strip != cached_strip) {
            cached_strip = strip;
            cached_base = -1;
            c0 = strip * F_COLS + lane * 8;
            const int64_t left = p.cols - c0;
            nvalid = left >= 8 ? 8 : (left > 0 ? (int)left : 0);
            if constexpr (NORM_COLS) {
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    sc[j] = j < nvalid ? scale_of(DASS_LD(&p.norm[c0 + j]), p.scale_mode, p.alpha) : 0.0f;
            }
        }
        if constexpr (!NORM_COLS) {
            const int64_t base = r0 & ~(int64_t)31;
            if (base != cached_base) {
                cached_base = base;
                const int64_t r = base + lane;
                lane_scale = r < p.rows ? scale_of(DASS_LD(&p.norm[r]), p.scale_mode, p.alpha) : 0.0f;
            }
        }

        // this unit's slab has landed once at most STAGES-2 younger groups are pending; then refill the
        // slot that was consumed one iteration ago with the unit STAGES-1 ahead
        cp_async_wait<STAGES - 2>();
        uint4 v[M];
#pragma unroll
        for (int q = 0; q < M; ++q) v[q] = *ring.slot(stage, q, lane);
        ring.issue(p, pre.strip, pre.g, u_pre < u_end, stage == 0 ? STAGES - 1 : stage - 1, lane);
        pre.advance(ups);
        ++u_pre;
        stage = stage + 1 == STAGES ? 0 : stage + 1;
        float rs[M];
#pragma unroll
        for (int q = 0; q < M; ++q) {
            rs[q] = 0.0f;
            if constexpr (!NORM_COLS) rs[q] = __shfl_sync(FULL_MASK, lane_scale, (int)(r0 & 31) + q);
        }

        // D[q]: bit j = "row q is pruned at column j" (the sign of p - t, t the column group's cut value)
        uint32_t D[M];
#pragma unroll
        for (int q = 0; q < M; ++q) D[q] = 0u;
        bool tie = false;
#pragma unroll
        for (int j = 7; j >= 0; --j) {       // column 7 first: after 8 inserts column j sits at bit j
            float pf[M];
#pragma unroll
            for (int q = 0; q < M; ++q) pf[q] = prod_of(word_of(v[q], j >> 1), (j & 1) != 0, NORM_COLS ? sc[j] : rs[q]);
            tie |= threshold_group<M>(pf, p.n_keep, D);
        }
        uint32_t K[M];
#pragma unroll
        for (int q = 0; q < M; ++q) K[q] = ~D[q];
        if (tie && nvalid > 0) {   // ragged lanes (zero padding ties) also land here; still exact
            TileWords<M> t;
            Scales8 s8;
#pragma unroll
            for (int q = 0; q < M; ++q) t.v[q] = v[q];
#pragma unroll
            for (int j = 0; j < 8; ++j) s8.s[j] = NORM_COLS ? sc[j] : (j < M ? rs[j < M ? j : 0] : 0.0f);
            const KeepWords<M> e = exact_keep_rows<M>(t, s8, NORM_COLS ? 1 : 0, p.n_keep);
#pragma unroll
            for (int q = 0; q < M; ++q) K[q] = e.k[q];
        }
        const uint32_t valid = (1u << nvalid) - 1u;
#pragma unroll
        for (int q = 0; q < M; ++q) {
            const uint32_t keep = K[q] & valid;
            const uint32_t word = quad_pack_bytes(keep, lane);
            if (p.mask && (lane & 3) == 0 && nvalid > 0) DASS_ST(&p.mask[(r0 + q) * p.wpr + (c0 >> 5)], word);
            if (p.Wp && nvalid > 0) {
                apply_keep_byte(v[q], keep);
                store_chunk(p.Wp + (r0 + q) * p.ld + c0, v[q], nvalid);
            }
        }
    }
}

// ---------------------------------------------------------------- groups along the columns (down)
// 3 CTAs per SM (85 registers): with 4 the 2:4 kernel spills a few words and runs 4 % slower
template <int M, bool NORM_COLS>
__global__ void __launch_bounds__(F_THREADS, 3) score_cols_bf16_kernel(const ScoreFastParams p)
{
    constexpr int G = 8 / M;             // groups inside a lane's 8 columns
    constexpr int STAGES = ring_stages(F_SLAB);
    extern __shared__ uint4 ring_mem[];
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (F_THREADS / 32) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (F_THREADS / 32);
    const int64_t u_begin = p.units * warp / nwarps;
    const int64_t u_end = p.units * (warp + 1) / nwarps;
    SlabRing<F_SLAB, STAGES> ring;
    ring.buf = ring_mem + (threadIdx.x >> 5) * (STAGES * F_SLAB * 32);
    const int ups = (int)p.units_per_strip;
    UnitCursor cur, pre;
    cur.strip = (int)(u_begin / p.units_per_strip);
    cur.g = (int)(u_begin - (int64_t)cur.strip * p.units_per_strip);
    pre = cur;
    int64_t u_pre = u_begin;
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        ring.issue(p, pre.strip, pre.g, u_pre < u_end, s, lane);
        pre.advance(ups);
        ++u_pre;
    }

    int64_t cached_strip = -1, cached_base = -1;
    float sc[8];
    float lane_scale = 0.0f;
    int nvalid = 0;
    int64_t c0 = 0;
    int stage = 0;

    for (int64_t u = u_begin; u < u_end; ++u, cur.advance(ups)) {
        const int64_t strip = cur.strip;
        const int64_t r0 = (int64_t)cur.g * F_SLAB;
        if (strip != cached_strip) {
            cached_strip = strip;
            cached_base = -1;
            c0 = strip * F_COLS + lane * 8;
            const int64_t left = p.cols - c0;
            nvalid = left >= 8 ? 8 : (left > 0 ? (int)left : 0);      // a multiple of M
            if constexpr (NORM_COLS) {
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    sc[j] = j < nvalid ? scale_of(DASS_LD(&p.norm[c0 + j]), p.scale_mode, p.alpha) : 0.0f;
            }
        }
        if constexpr (!NORM_COLS) {
            const int64_t base = r0 & ~(int64_t)31;
            if (base != cached_base) {
                cached_base = base;
                const int64_t r = base + lane;
                lane_scale = r < p.rows ? scale_of(DASS_LD(&p.norm[r]), p.scale_mode, p.alpha) : 0.0f;
            }
        }

        cp_async_wait<STAGES - 2>();
        uint4 v[F_SLAB];
#pragma unroll
        for (int i = 0; i < F_SLAB; ++i) v[i] = *ring.slot(stage, i, lane);
        ring.issue(p, pre.strip, pre.g, u_pre < u_end, stage == 0 ? STAGES - 1 : stage - 1, lane);
        pre.advance(ups);
        ++u_pre;
        stage = stage + 1 == STAGES ? 0 : stage + 1;

        // Every group is compared with its own cut value t (the n_keep-th largest rounded product): the sign of
        // p - t is shifted straight into the row's byte, column 7 first, so that bit j ends up as "column j pruned".
        // The rule is proven unless t equals the next value (a tie across the cut): then the slab goes the exact way.
        uint32_t row_keep[F_SLAB];
        bool tie = false;
        float rsv[F_SLAB];
#pragma unroll
        for (int i = 0; i < F_SLAB; ++i) {
            float rs = 0.0f;
            if constexpr (!NORM_COLS) rs = __shfl_sync(FULL_MASK, lane_scale, (int)(r0 & 31) + i);
            rsv[i] = rs;
            uint32_t pruned = 0u;
#pragma unroll
            for (int g = G - 1; g >= 0; --g) {
                float pf[M];
#pragma unroll
                for (int q = 0; q < M; ++q) {
                    const int j = g * M + q;
                    pf[q] = prod_of(word_of(v[i], j >> 1), (j & 1) != 0, NORM_COLS ? sc[j] : rs);
                }
                float t, next;
                cut_values<M>(pf, p.n_keep, t, next);
                tie |= t == next;
#pragma unroll
                for (int q = M - 1; q >= 0; --q) pruned = __funnelshift_l(__float_as_uint(__fsub_rn(pf[q], t)), pruned, 1);
            }
            row_keep[i] = ~pruned & 0xffu;
        }
        if (tie && nvalid > 0) {   // ragged slabs (zero padding ties) also land here; still exact
            TileWords<F_SLAB> t;
            Scales8 s8;
#pragma unroll
            for (int i = 0; i < F_SLAB; ++i) t.v[i] = v[i];
#pragma unroll
            for (int i = 0; i < 8; ++i) s8.s[i] = NORM_COLS ? sc[i] : (i < F_SLAB ? rsv[i < F_SLAB ? i : 0] : 0.0f);
            const KeepWords<F_SLAB> e = exact_keep_cols<M>(t, s8, NORM_COLS ? 1 : 0, p.n_keep);
#pragma unroll
            for (int i = 0; i < F_SLAB; ++i) row_keep[i] = e.k[i];
        }
        const uint32_t valid = (1u << nvalid) - 1u;
#pragma unroll
        for (int i = 0; i < F_SLAB; ++i) {
            const uint32_t keep = row_keep[i] & valid;
            const uint32_t word = quad_pack_bytes(keep, lane);
            if (r0 + i < p.rows && nvalid > 0) {
                if (p.mask && (lane & 3) == 0) DASS_ST(&p.mask[(r0 + i) * p.wpr + (c0 >> 5)], word);
                if (p.Wp) {
                    apply_keep_byte(v[i], keep);
                    store_chunk(p.Wp + (r0 + i) * p.ld + c0, v[i], nvalid);
                }
            }
        }
    }
}

int device_sm_count();   // dass_abi.cu

template <typename K>
static cudaError_t launch_with_ring(K kernel, int smem, const ScoreFastParams &p, int grid, cudaStream_t st)
{
    if (smem > 48 * 1024) {
        const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
    }
    kernel<<<grid, F_THREADS, smem, st>>>(p);
    return cudaGetLastError();
}

template <int M>
static cudaError_t launch_fast(const ScoreFastParams &p, bool norm_cols, bool group_cols, int grid, cudaStream_t st)
{
    if (group_cols) {
        constexpr int smem = ring_bytes(F_SLAB);
        return norm_cols ? launch_with_ring(score_cols_bf16_kernel<M, true>, smem, p, grid, st)
                         : launch_with_ring(score_cols_bf16_kernel<M, false>, smem, p, grid, st);
    }
    constexpr int smem = ring_bytes(M);
    return norm_cols ? launch_with_ring(score_rows_bf16_kernel<M, true>, smem, p, grid, st)
                     : launch_with_ring(score_rows_bf16_kernel<M, false>, smem, p, grid, st);
}

cudaError_t score_nm_bf16_launch(const void *W, int64_t rows, int64_t cols, int64_t ld,
                                 const float *norm, bool norm_cols, float alpha, int n_keep, int m, bool group_cols,
                                 uint32_t *mask_bits, void *W_pruned, cudaStream_t st)
{
    ScoreFastParams p;
    p.W = static_cast<const uint16_t *>(W);
    p.Wp = static_cast<uint16_t *>(W_pruned);
    p.mask = mask_bits; p.norm = norm;
    p.rows = rows; p.cols = cols; p.ld = ld;
    p.wpr = (cols + 31) / 32;
    const int64_t strips = (cols + F_COLS - 1) / F_COLS;
    p.units_per_strip = group_cols ? (rows + F_SLAB - 1) / F_SLAB : rows / m;
    p.units = strips * p.units_per_strip;
    p.n_keep = n_keep;
    p.scale_mode = (int)scale_mode_for(alpha);
    p.alpha = alpha;
    const int64_t wpb = F_THREADS / 32;
    const int64_t want = (p.units + wpb - 1) / wpb;
    const int64_t cap = (int64_t)device_sm_count() * 8;
    const int grid = (int)(want < cap ? want : cap);
    return m == 4 ? launch_fast<4>(p, norm_cols, group_cols, grid, st) : launch_fast<8>(p, norm_cols, group_cols, grid, st);
}

}  // namespace dass
