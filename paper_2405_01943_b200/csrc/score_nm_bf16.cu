// Stage (b) for bf16 weights: Eq. 4 / Eq. 5 score and N:M selection, tuned to stay under the HBM roofline.
//
// Same tiling as the generic kernels in score_nm.cu (a lane owns 8 consecutive columns = one 16-byte
// vector; a warp row is one contiguous 512-byte segment), but the selection is done with 32-bit
// integer and bit-sliced logic instead of per-element double arithmetic:
//
//   * p = fl32(|w| * scale).  Rounding is monotone, so p_b > p_a proves score_b > score_a for the
//     exact products; non-negative floats order like their bit patterns, so the comparison is the
//     sign of an integer subtraction, shifted into a bit-sliced word with one funnel shift (bit j of a
//     word = column j, or row j, of the lane's tile).
//   * ranks are counted with full adders on those words (one LOP3 each) and compared with n_keep, which
//     yields the keep bits of 8 groups at once;
//   * only when two rounded products of a group are EQUAL is the order not proven; the lane then
//     recomputes its tile's keep bits with exact double products (rare on real data, always correct).
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
#ifndef F_MIN_BLOCKS
#define F_MIN_BLOCKS 4
#endif
constexpr int F_COLS = 256;          // columns per warp strip
#ifndef F_SLAB_ROWS
#define F_SLAB_ROWS 4
#endif
constexpr int F_SLAB = F_SLAB_ROWS;  // rows per unit when groups run along the columns (4 or 8)

// Out of line on purpose: the double-precision sqrt / pow sequences would otherwise inflate the register
// budget of the streaming loops, and they run once per strip or per 32 rows only.
__device__ __noinline__ float scale_of(float n, int mode, float alpha) { return scale_from_norm(n, mode, alpha); }

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// bits of fl32(|element| * scale); element = low (hi == false) or high half of a word of two bf16
__device__ __forceinline__ uint32_t prod_bits(uint32_t word, bool hi, float scale)
{
    const uint32_t fb = hi ? (word & 0xffff0000u) : (word << 16);
    return __float_as_uint(fabsf(__uint_as_float(fb)) * scale);
}

// full adder on bit-sliced words
__device__ __forceinline__ uint32_t xor3(uint32_t a, uint32_t b, uint32_t c) { return a ^ b ^ c; }
__device__ __forceinline__ uint32_t maj3(uint32_t a, uint32_t b, uint32_t c) { return (a & b) | (a & c) | (b & c); }

// rank < n_keep for a bit-sliced 3-bit rank (b2 b1 b0), n_keep in 1..7
__device__ __forceinline__ uint32_t rank_below(uint32_t b2, uint32_t b1, uint32_t b0, int n_keep)
{
    switch (n_keep) {
    case 1: return ~(b2 | b1 | b0);
    case 2: return ~(b2 | b1);
    case 3: return ~(b2 | (b1 & b0));
    case 4: return ~b2;
    case 5: return ~(b2 & (b1 | b0));
    case 6: return ~(b2 & b1);
    default: return ~(b2 & b1 & b0);
    }
}

// Pair index of (a, b), a < b, in the order (0,1),(0,2),...,(0,M-1),(1,2),...
template <int M>
__host__ __device__ constexpr int pair_index(int a, int b) { return a * M - a * (a + 1) / 2 + (b - a - 1); }

// Keep words from the bit-sliced comparison words C[pair] (bit set: the later element b beats a).
// Element a is preceded by every earlier k that b-beats... i.e. rank_a = sum_{k<a} !C[k,a] + sum_{k>a} C[a,k].
template <int M>
__device__ __forceinline__ void keep_from_pairs(const uint32_t (&C)[M * (M - 1) / 2], int n_keep, uint32_t (&K)[M])
{
#pragma unroll
    for (int a = 0; a < M; ++a) {
        uint32_t in[M - 1];
#pragma unroll
        for (int k = 0; k < M; ++k) {
            if (k < a) in[k] = ~C[pair_index<M>(k, a)];
            else if (k > a) in[k - 1] = C[pair_index<M>(a, k)];
        }
        if constexpr (M == 4) {
            const uint32_t b0 = xor3(in[0], in[1], in[2]);
            const uint32_t b1 = maj3(in[0], in[1], in[2]);
            K[a] = rank_below(0u, b1, b0, n_keep);
        } else {
            const uint32_t s1 = xor3(in[0], in[1], in[2]), c1 = maj3(in[0], in[1], in[2]);
            const uint32_t s2 = xor3(in[3], in[4], in[5]), c2 = maj3(in[3], in[4], in[5]);
            const uint32_t b0 = xor3(s1, s2, in[6]), c3 = maj3(s1, s2, in[6]);
            const uint32_t b1 = xor3(c1, c2, c3), b2 = maj3(c1, c2, c3);
            K[a] = rank_below(b2, b1, b0, n_keep);
        }
    }
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
        __stcs(reinterpret_cast<uint4 *>(dst), v);
    } else {
        for (int j = 0; j < nvalid; ++j) {
            const uint32_t w = word_of(v, j >> 1);
            dst[j] = (uint16_t)((j & 1) ? (w >> 16) : (w & 0xffffu));
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
__global__ void __launch_bounds__(F_THREADS, F_MIN_BLOCKS) score_rows_bf16_kernel(const ScoreFastParams p)
{
    constexpr int NP = M * (M - 1) / 2;
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (F_THREADS / 32) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (F_THREADS / 32);
    const int64_t u_begin = p.units * warp / nwarps;
    const int64_t u_end = p.units * (warp + 1) / nwarps;

    int64_t cached_strip = -1, cached_base = -1;
    float sc[8];          // per-column scales of the strip (NORM_COLS)
    float lane_scale = 0.0f;   // scale of row cached_base + lane (!NORM_COLS)
    int nvalid = 0;
    int64_t c0 = 0;

    for (int64_t u = u_begin; u < u_end; ++u) {
        const int64_t strip = u / p.units_per_strip;
        const int64_t r0 = (u - strip * p.units_per_strip) * M;
        if (strip != cached_strip) {
            cached_strip = strip;
            cached_base = -1;
            c0 = strip * F_COLS + lane * 8;
            const int64_t left = p.cols - c0;
            nvalid = left >= 8 ? 8 : (left > 0 ? (int)left : 0);
            if constexpr (NORM_COLS) {
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    sc[j] = j < nvalid ? scale_of(p.norm[c0 + j], p.scale_mode, p.alpha) : 0.0f;
            }
        }
        if constexpr (!NORM_COLS) {
            const int64_t base = r0 & ~(int64_t)31;
            if (base != cached_base) {
                cached_base = base;
                const int64_t r = base + lane;
                lane_scale = r < p.rows ? scale_of(p.norm[r], p.scale_mode, p.alpha) : 0.0f;
            }
        }

        uint4 v[M];
#pragma unroll
        for (int q = 0; q < M; ++q) {
            if (nvalid > 0) v[q] = __ldcs(reinterpret_cast<const uint4 *>(p.W + (r0 + q) * p.ld + c0));
            else v[q] = make_uint4(0u, 0u, 0u, 0u);
        }
        float rs[M];
#pragma unroll
        for (int q = 0; q < M; ++q) {
            rs[q] = 0.0f;
            if constexpr (!NORM_COLS) rs[q] = __shfl_sync(FULL_MASK, lane_scale, (int)(r0 & 31) + q);
        }

        uint32_t C[NP];
#pragma unroll
        for (int i = 0; i < NP; ++i) C[i] = 0u;
        bool tie = false;
#pragma unroll
        for (int j = 7; j >= 0; --j) {       // column 7 first: after 8 inserts column j sits at bit j
            uint32_t pb[M];
#pragma unroll
            for (int q = 0; q < M; ++q) pb[q] = prod_bits(word_of(v[q], j >> 1), (j & 1) != 0, NORM_COLS ? sc[j] : rs[q]);
#pragma unroll
            for (int a = 0; a < M; ++a)
#pragma unroll
                for (int b = a + 1; b < M; ++b) {
                    const uint32_t dlt = pb[a] - pb[b];                     // negative iff p_b > p_a
                    C[pair_index<M>(a, b)] = __funnelshift_l(dlt, C[pair_index<M>(a, b)], 1);
                    tie |= (dlt == 0u);
                }
        }
        uint32_t K[M];
        keep_from_pairs<M>(C, p.n_keep, K);
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
            if (p.mask && (lane & 3) == 0 && nvalid > 0) p.mask[(r0 + q) * p.wpr + (c0 >> 5)] = word;
            if (p.Wp && nvalid > 0) {
                apply_keep_byte(v[q], keep);
                store_chunk(p.Wp + (r0 + q) * p.ld + c0, v[q], nvalid);
            }
        }
    }
}

// ---------------------------------------------------------------- groups along the columns (down)
template <int M, bool NORM_COLS>
__global__ void __launch_bounds__(F_THREADS, F_MIN_BLOCKS) score_cols_bf16_kernel(const ScoreFastParams p)
{
    constexpr int NP = M * (M - 1) / 2;
    constexpr int G = 8 / M;             // groups inside a lane's 8 columns
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (F_THREADS / 32) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (F_THREADS / 32);
    const int64_t u_begin = p.units * warp / nwarps;
    const int64_t u_end = p.units * (warp + 1) / nwarps;

    int64_t cached_strip = -1, cached_base = -1;
    float sc[8];
    float lane_scale = 0.0f;
    int nvalid = 0;
    int64_t c0 = 0;

    for (int64_t u = u_begin; u < u_end; ++u) {
        const int64_t strip = u / p.units_per_strip;
        const int64_t r0 = (u - strip * p.units_per_strip) * F_SLAB;
        if (strip != cached_strip) {
            cached_strip = strip;
            cached_base = -1;
            c0 = strip * F_COLS + lane * 8;
            const int64_t left = p.cols - c0;
            nvalid = left >= 8 ? 8 : (left > 0 ? (int)left : 0);      // a multiple of M
            if constexpr (NORM_COLS) {
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    sc[j] = j < nvalid ? scale_of(p.norm[c0 + j], p.scale_mode, p.alpha) : 0.0f;
            }
        }
        if constexpr (!NORM_COLS) {
            const int64_t base = r0 & ~(int64_t)31;
            if (base != cached_base) {
                cached_base = base;
                const int64_t r = base + lane;
                lane_scale = r < p.rows ? scale_of(p.norm[r], p.scale_mode, p.alpha) : 0.0f;
            }
        }

        uint4 v[F_SLAB];
#pragma unroll
        for (int i = 0; i < F_SLAB; ++i) {
            if (nvalid > 0 && r0 + i < p.rows) v[i] = __ldcs(reinterpret_cast<const uint4 *>(p.W + (r0 + i) * p.ld + c0));
            else v[i] = make_uint4(0u, 0u, 0u, 0u);
        }

        uint32_t C[G][NP];
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int i = 0; i < NP; ++i) C[g][i] = 0u;
        bool tie = false;
        float rsv[F_SLAB];
#pragma unroll
        for (int i = F_SLAB - 1; i >= 0; --i) {       // row 7 first: after 8 inserts row i sits at bit i
            float rs = 0.0f;
            if constexpr (!NORM_COLS) rs = __shfl_sync(FULL_MASK, lane_scale, (int)(r0 & 31) + i);
            rsv[i] = rs;
#pragma unroll
            for (int g = 0; g < G; ++g) {
                uint32_t pb[M];
#pragma unroll
                for (int q = 0; q < M; ++q) {
                    const int j = g * M + q;
                    pb[q] = prod_bits(word_of(v[i], j >> 1), (j & 1) != 0, NORM_COLS ? sc[j] : rs);
                }
#pragma unroll
                for (int a = 0; a < M; ++a)
#pragma unroll
                    for (int b = a + 1; b < M; ++b) {
                        const uint32_t dlt = pb[a] - pb[b];
                        C[g][pair_index<M>(a, b)] = __funnelshift_l(dlt, C[g][pair_index<M>(a, b)], 1);
                        tie |= (dlt == 0u);
                    }
            }
        }
        // Q[h]: byte a = keep bits (bit i = row i) of column 4h + a
        uint32_t Q[2];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            uint32_t K[M];
            keep_from_pairs<M>(C[g], p.n_keep, K);
#pragma unroll
            for (int h = 0; h < M / 4; ++h) {
                const uint32_t q = (K[4 * h] & 0xffu) | ((K[4 * h + 1] & 0xffu) << 8) | ((K[4 * h + 2] & 0xffu) << 16) |
                                   (K[4 * h + 3] << 24);
                Q[g * (M / 4) + h] = q;
            }
        }
        uint32_t row_keep[F_SLAB];
#pragma unroll
        for (int i = 0; i < F_SLAB; ++i) {
            // gather bit i of each byte of Q[h] into a nibble (columns 4h .. 4h+3)
            const uint32_t n0 = (((Q[0] >> i) & 0x01010101u) * 0x10204080u) >> 28;
            const uint32_t n1 = (((Q[1] >> i) & 0x01010101u) * 0x10204080u) >> 28;
            row_keep[i] = n0 | (n1 << 4);
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
                if (p.mask && (lane & 3) == 0) p.mask[(r0 + i) * p.wpr + (c0 >> 5)] = word;
                if (p.Wp) {
                    apply_keep_byte(v[i], keep);
                    store_chunk(p.Wp + (r0 + i) * p.ld + c0, v[i], nvalid);
                }
            }
        }
    }
}

int device_sm_count();   // dass_abi.cu

template <int M>
static cudaError_t launch_fast(const ScoreFastParams &p, bool norm_cols, bool group_cols, int grid, cudaStream_t st)
{
    if (group_cols) {
        if (norm_cols) score_cols_bf16_kernel<M, true><<<grid, F_THREADS, 0, st>>>(p);
        else score_cols_bf16_kernel<M, false><<<grid, F_THREADS, 0, st>>>(p);
    } else {
        if (norm_cols) score_rows_bf16_kernel<M, true><<<grid, F_THREADS, 0, st>>>(p);
        else score_rows_bf16_kernel<M, false><<<grid, F_THREADS, 0, st>>>(p);
    }
    return cudaGetLastError();
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
