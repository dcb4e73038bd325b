// Unstructured selection, lines that are matrix columns: the streaming passes that apply the per-column results of
// select_cols_kernel to the matrix (mask words and pruned copy, coalesced rows), and the kernel that ranks what the
// bf16 pass set aside.
#include "select_common.cuh"

namespace dass {

// ---------------------------------------------------------------- column lines: streaming emit
// Applies the per-column thresholds to the matrix with the tiling of the N:M kernels (a lane owns 8 consecutive
// columns, a warp row is 512 contiguous bytes), so the mask words and the pruned copy are written coalesced.
struct EmitParams {
    const void *W;
    void *Wp;
    uint32_t *mask;
    const float *scale;
    const LineResult *results;   // one per column
    int64_t rows, cols, ld, wpr;
    int64_t col_blocks, row_blocks;
    int scale_per_row;           // 1: scale[r] (the norm runs along the lines), 0: scale[c]
};

// Rare path of the emit pass, kept out of line so that the streaming loop stays small enough to unroll: the
// element's rounded product equals a threshold that the exact stage had to split.
__device__ __noinline__ bool exact_tie_keeps(const LineResult *res, float a, float s, int64_t r)
{
    const unsigned long long k64 = (unsigned long long)__double_as_longlong((double)a * (double)s);
    const LineResult t = DASS_LD(res);
    return k64 > t.tau64 || (k64 == t.tau64 && (long long)r <= t.cut);
}

template <bool BF16>
__global__ void __launch_bounds__(256, 4) select_emit_cols_kernel(const EmitParams p)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * 8;
    const int64_t ntasks = p.col_blocks * p.row_blocks;
    for (int64_t task = warp; task < ntasks; task += nwarps) {
        const int64_t cb = task % p.col_blocks, rb = task / p.col_blocks;
        const int64_t c0 = cb * 256 + lane * 8;
        const int64_t left = p.cols - c0;
        const int nvalid = left >= 8 ? 8 : (left > 0 ? (int)left : 0);
        uint32_t tau[8];
        float sc[8];
        uint32_t exact_cols = 0u;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            tau[j] = 0xffffffffu;
            sc[j] = 0.0f;
            if (j < nvalid) {
                tau[j] = DASS_LD(&p.results[c0 + j].tau32);
                exact_cols |= (DASS_LD(&p.results[c0 + j].exact) ? 1u : 0u) << j;
                if (!p.scale_per_row) sc[j] = DASS_LD(&p.scale[c0 + j]);
            }
        }
        if ((cb + 1) * 256 > p.cols) {
            // the ragged last strip: row by row
            for (int i = 0; i < 32; ++i) {
                const int64_t r = rb * 32 + i;
                if (r >= p.rows) break;                     // warp-uniform
                Chunk<BF16> ch;
                if (nvalid > 0) chunk_load<BF16>(ch, p.W, r * p.ld + c0, nvalid);
                else chunk_zero<BF16>(ch);
                const float rs = p.scale_per_row ? DASS_LD_G(p.scale + r) : 0.0f;
                uint32_t keep = 0u;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float a = chunk_abs<BF16>(ch, j);
                    const float s = p.scale_per_row ? rs : sc[j];
                    const uint32_t key = __float_as_uint(__fmul_rn(a, s));
                    bool k = key > tau[j];
                    if (key == tau[j] && j < nvalid) {
                        k = true;                           // products equal to the threshold stay ...
                        if ((exact_cols >> j) & 1u) {       // ... unless the exact stage had to split them
                            const LineResult res = DASS_LD(&p.results[c0 + j]);
                            const unsigned long long k64 = (unsigned long long)__double_as_longlong((double)a * (double)s);
                            k = k64 > res.tau64 || (k64 == res.tau64 && (long long)r <= res.cut);
                        }
                    }
                    keep |= (k && j < nvalid ? 1u : 0u) << j;
                }
                const uint32_t word = quad_pack_bytes(keep, lane);
                if (nvalid > 0) {
                    if (p.mask && (lane & 3) == 0) DASS_ST(&p.mask[r * p.wpr + (c0 >> 5)], word);
                    if (p.Wp) {
                        chunk_apply_mask<BF16>(ch, keep);
                        chunk_store<BF16>(ch, p.Wp, r * p.ld + c0, nvalid);
                    }
                }
            }
            continue;
        }
        // whole strips, 4 rows at a time: all their loads are issued before any row is processed (measured: 4 CTAs
        // per SM with batches of 4 rows beat 2 CTAs with batches of 8 and 5 CTAs with their spills)
#pragma unroll 1
        for (int i0 = 0; i0 < 32; i0 += 4) {
            const int64_t rbase = rb * 32 + i0;
            if (rbase >= p.rows) break;                     // warp-uniform
            Chunk<BF16> chs[4];
            float rss[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int64_t r = rbase + u;
                if (r < p.rows) chunk_load<BF16>(chs[u], p.W, r * p.ld + c0, 8);
                else chunk_zero<BF16>(chs[u]);
                rss[u] = (p.scale_per_row && r < p.rows) ? DASS_LD_G(p.scale + r) : 0.0f;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int64_t r = rbase + u;
                uint32_t keep = 0u;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float a = chunk_abs<BF16>(chs[u], j);
                    const float s = p.scale_per_row ? rss[u] : sc[j];
                    const uint32_t key = __float_as_uint(__fmul_rn(a, s));
                    bool k = key >= tau[j];                 // products equal to the threshold stay ...
                    if (key == tau[j] && ((exact_cols >> j) & 1u))
                        k = exact_tie_keeps(p.results + c0 + j, a, s, r);   // ... unless the exact stage split them
                    keep |= (k ? 1u : 0u) << j;
                }
                const uint32_t word = quad_pack_bytes(keep, lane);
                if (r < p.rows) {
                    if (p.mask && (lane & 3) == 0) DASS_ST(&p.mask[r * p.wpr + (c0 >> 5)], word);
                    if (p.Wp) {
                        chunk_apply_mask<BF16>(chs[u], keep);
                        if constexpr (BF16) {
                            DASS_ST_CS(reinterpret_cast<uint4 *>(static_cast<uint16_t *>(p.Wp) + r * p.ld + c0),
                                   make_uint4(chs[u].w[0], chs[u].w[1], chs[u].w[2], chs[u].w[3]));
                        } else {
                            uint4 *dst = reinterpret_cast<uint4 *>(static_cast<uint32_t *>(p.Wp) + r * p.ld + c0);
                            DASS_ST_CS(dst, make_uint4(chs[u].w[0], chs[u].w[1], chs[u].w[2], chs[u].w[3]));
                            DASS_ST_CS(dst + 1, make_uint4(chs[u].w[4], chs[u].w[5], chs[u].w[6], chs[u].w[7]));
                        }
                    }
                }
            }
        }
    }
}

// ---------------------------------------------------------------- column lines, bf16: streaming emit fed by TMA
// The same job with the machinery of the one-pass N:M kernels (stream_units.cuh): 8 x 256 units arrive through a
// per-warp ring of TMA boxes, a warp walks down a strip so that a lane's 8 columns -- and with them its thresholds --
// stay the same for the whole run, and "product < threshold" is read off the sign of a float difference that one
// byte permute turns into the pruned-lane mask of a word.  Columns whose threshold the exact stage had to split
// (rounded products tie across the cut) take a scalar fix-up for the elements equal to the threshold.
constexpr int SE_MIN_BLOCKS = 5;                 // CTAs per SM the emit kernel is built for
constexpr int SE_STAGES = 2;                     // ring slots per warp (a third slot would cost the fifth CTA its shared memory)
struct EmitStreamParams : UnitGrid {
    const uint16_t *W;
    uint16_t *Wp;        // nullable
    uint32_t *mask;      // nullable
    const float *scale;
    const LineResult *results;
    CandLists cand;
    int64_t ld, wpr;
    int scale_per_row;
};

// Rare path of the emit pass: the elements of one row of a lane's tile that lie in their column's undecided bin are
// appended to that column's list (they were written as pruned; the ranking kernel brings the survivors back).
__device__ __noinline__ void emit_set_aside(uint4 row, uint32_t in_bin, const float *col_scales, float row_scale,
                                            int scale_per_row, long long r, long long c0, CandLists cl)
{
    while (in_bin) {
        const int j = __ffs((int)in_bin) - 1;
        in_bin &= in_bin - 1u;
        const uint32_t w = wsel(row, j >> 1);
        const uint32_t raw = (j & 1) ? (w & 0xffff0000u) : (w << 16);
        const float s = scale_per_row ? row_scale : DASS_LD(&col_scales[c0 + j]);
        const uint32_t key = __float_as_uint(fabsf(__uint_as_float(raw)) * s);
        const uint32_t slot = atomicAdd(cl.count + c0 + j, 1u);
        if (slot < (uint32_t)CAND_CAP) {
            const size_t at = (size_t)(c0 + j) * CAND_CAP + slot;
            DASS_ST(&cl.key[at], key);
            DASS_ST(&cl.idx[at], (uint32_t)r);
            DASS_ST(&cl.raw[at], raw);
        }
    }
}

// Keep byte of one row of a lane's tile when some of its columns need the exact rule (rare).
__device__ __noinline__ uint32_t emit_exact_row(uint4 row, uint32_t keep, uint32_t exact_cols, const LineResult *res8,
                                                const float *col_scales8, float row_scale, int scale_per_row, long long r)
{
    while (exact_cols) {
        const int j = __ffs((int)exact_cols) - 1;
        exact_cols &= exact_cols - 1u;
        const uint32_t w = wsel(row, j >> 1);
        const float a = fabsf(__uint_as_float((j & 1) ? (w & 0xffff0000u) : (w << 16)));
        const float s = scale_per_row ? row_scale : DASS_LD(&col_scales8[j]);
        const LineResult t = DASS_LD(res8 + j);
        if (__float_as_uint(__fmul_rn(a, s)) != t.tau32) continue;          // only products equal to the threshold
        const unsigned long long k64 = (unsigned long long)__double_as_longlong((double)a * (double)s);
        const bool k = k64 > t.tau64 || (k64 == t.tau64 && r <= t.cut);
        keep = (keep & ~(1u << j)) | ((k ? 1u : 0u) << j);
    }
    return keep;
}

// PER_ROW: the scale belongs to the row (it varies down a column) rather than to the column.
template <bool PER_ROW>
__global__ void __launch_bounds__(PN_THREADS, SE_MIN_BLOCKS)
select_emit_stream_kernel(const __grid_constant__ CUtensorMap map_w, const EmitStreamParams p)
{
    extern __shared__ uint8_t se_smem_raw[];
    uint8_t *smem = se_smem_raw + ((128u - (smem_u32(se_smem_raw) & 127u)) & 127u);
    const int lane = threadIdx.x & 31;
    const uint32_t sel1 = (lane & 1) ? 0x3715u : 0x6240u;
    const uint32_t sel2 = (lane & 2) ? 0x3276u : 0x5410u;
    Run<true> run;                                   // down a strip: the lane's columns stay
    run.set(p, threadIdx.x >> 5);
    const int64_t c0 = (int64_t)run.line * PN_COLS + lane * 8;
    const int64_t left = p.cols - c0;
    const int nvalid = left >= 8 ? 8 : (left > 0 ? (int)left : 0);
    const uint32_t valid = (1u << nvalid) - 1u;
    const bool quad_live = (c0 & ~(int64_t)31) < p.cols;
    float tau[8], tlo[8], sc[8];                     // tlo: start of the column's undecided bin (none: infinity)
    uint32_t exact_cols = 0u, bin_cols = 0u;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        tau[j] = 0.0f;
        tlo[j] = __uint_as_float(0x7f800000u);
        sc[j] = 0.0f;
        if (j < nvalid) {
            tau[j] = __uint_as_float(DASS_LD(&p.results[c0 + j].tau32));
            const uint32_t mode = DASS_LD(&p.results[c0 + j].exact);
            exact_cols |= (mode == 1u ? 1u : 0u) << j;
            if (mode == LINE_BIN) {
                bin_cols |= 1u << j;
                tlo[j] = __uint_as_float((uint32_t)DASS_LD(&p.results[c0 + j].tau64));
            }
            if (!PER_ROW) sc[j] = DASS_LD(&p.scale[c0 + j]);
        }
    }
    const bool cols_full = __all_sync(FULL_MASK, nvalid == 8);     // the warp's 256 columns all exist
    UnitRing<true, SE_STAGES> ring;
    ring.start(smem, threadIdx.x >> 5, &map_w, p, run, lane);

    for (int f = run.f0; f < run.f1; ++f) {
        const uint4 *tile = ring.next(&map_w, p, run, lane);
        if (tile == nullptr) { ring.fail(lane, p.status); return; }
        const int64_t r0 = (int64_t)f * PN_ROWS;
        float rs[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) rs[i] = 0.0f;
        if constexpr (PER_ROW) {     // the scale vector is padded with zeros to a multiple of 8 and 32-byte aligned
            const float4 a = DASS_LD_G(reinterpret_cast<const float4 *>(p.scale + r0));
            const float4 b = DASS_LD_G(reinterpret_cast<const float4 *>(p.scale + r0) + 1);
            rs[0] = a.x; rs[1] = a.y; rs[2] = a.z; rs[3] = a.w; rs[4] = b.x; rs[5] = b.y; rs[6] = b.z; rs[7] = b.w;
        }
        // four rows of the tile; FULL: all four rows and all of the warp's columns lie inside the matrix
        auto four_rows = [&](auto full_tag, int h) {
            constexpr bool FULL = decltype(full_tag)::value;
            const int64_t rh = r0 + 4 * h;
            const int nrows = FULL ? 4 : (p.rows - rh >= 4 ? 4 : (int)(p.rows - rh));
            uint4 v[4];
            uint32_t Z[4][4];
            uint32_t aside[4];                       // per row: lanes below the threshold but not below the bin's start
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                v[i] = tile[(4 * h + i) * p.pitch16 + lane];
                aside[i] = 0u;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint32_t w = wsel(v[i], k);
                    const float pe = prod_lo(w, PER_ROW ? rs[4 * h + i] : sc[2 * k]);
                    const float po = prod_hi(w, PER_ROW ? rs[4 * h + i] : sc[2 * k + 1]);
                    Z[i][k] = pruned_lanes(__fsub_rn(pe, tau[2 * k]), __fsub_rn(po, tau[2 * k + 1]));
                    aside[i] |= Z[i][k] & ~pruned_lanes(__fsub_rn(pe, tlo[2 * k]), __fsub_rn(po, tlo[2 * k + 1])) & (0x00010001u << (2 * k));
                }
            }
            uint32_t keep = ~bytes_of_lanes4(Z[0], Z[1], Z[2], Z[3]);
            if constexpr (!FULL) keep &= (valid * 0x01010101u) & (nrows == 4 ? 0xffffffffu : ((1u << (8 * nrows)) - 1u));
            if (aside[0] | aside[1] | aside[2] | aside[3]) {     // elements of undecided bins: set aside for the ranking
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t in_bin = (aside[i] | (aside[i] >> 15)) & (FULL ? 0xffu : valid) & bin_cols;   // bit j = column j
                    if (i < nrows && in_bin)
                        emit_set_aside(v[i], in_bin, p.scale, rs[4 * h + i], PER_ROW ? 1 : 0, (long long)(rh + i), c0, p.cand);
                }
            }
            if (exact_cols) {                        // rounded products equal to a split threshold: the exact rule decides
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (i < nrows) {
                        const uint32_t kb = emit_exact_row(v[i], (keep >> (8 * i)) & 0xffu, exact_cols, p.results + c0, p.scale + c0,
                                                           rs[4 * h + i], PER_ROW ? 1 : 0, (long long)(rh + i));
                        keep = (keep & ~(0xffu << (8 * i))) | (kb << (8 * i));
                        uint32_t m[4];
                        lanes_of_byte(kb, m);
#pragma unroll
                        for (int k = 0; k < 4; ++k) Z[i][k] = ~m[k];
                    }
                }
            }
            const bool row_live = FULL || (lane & 3) < nrows;
            if (p.mask) {
                const uint32_t word = quad_transpose(keep, sel1, sel2);
                if ((FULL || quad_live) && row_live) DASS_ST(&p.mask[(rh + (lane & 3)) * p.wpr + (c0 >> 5)], word);
            }
            if (p.Wp && (FULL || nvalid > 0)) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (i < nrows) {
                        uint4 P;
#pragma unroll
                        for (int k = 0; k < 4; ++k) wref(P, k) = wsel(v[i], k) & ~Z[i][k];
                        store_row8(p.Wp + (rh + i) * p.ld + c0, P, FULL ? 8 : nvalid);
                    }
                }
            }
        };
        if (cols_full && r0 + PN_ROWS <= p.rows) {   // warp-uniform: the common tile
#pragma unroll
            for (int h = 0; h < PN_ROWS / 4; ++h) four_rows(std::true_type{}, h);
        } else {
#pragma unroll
            for (int h = 0; h < PN_ROWS / 4; ++h)
                if (r0 + 4 * h < p.rows) four_rows(std::false_type{}, h);
        }
    }
}

// ---------------------------------------------------------------- column lines: the undecided bins
// One warp per column that the selection left at a bin: the elements the emit pass set aside are ranked by the full
// key (rounded product, exact product, lower row first), the column's rule is completed, and the survivors are put
// back into the mask and the pruned copy.
constexpr int FIX_WARPS = 8;
struct FixParams {
    LineResult *results;
    CandLists cand;
    const float *scale;
    uint16_t *Wp;        // nullable
    uint32_t *mask;      // nullable
    int64_t cols, ld, wpr;
    int scale_per_row;
    int *status;
};

__global__ void __launch_bounds__(FIX_WARPS * 32) select_fix_cols_kernel(const FixParams p)
{
    __shared__ CandSet cand[FIX_WARPS];
    __shared__ FastLine fl[FIX_WARPS];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t col = (int64_t)blockIdx.x * FIX_WARPS + w;
    if (col >= p.cols) return;
    const LineResult r = DASS_LD(&p.results[col]);
    if (r.exact != LINE_BIN) return;                 // warp-uniform
    const uint32_t n = DASS_LD(&p.cand.count[col]);
    const uint32_t bucket = (uint32_t)r.cut;
    if (n != bucket || n > (uint32_t)CAND_CAP) {     // the two passes disagree: cannot happen, is reported
        if (lane == 0) atomicMax(p.status, (int)DASS_ERR_INTERNAL);
        return;
    }
    const float col_scale = p.scale_per_row ? 0.0f : DASS_LD(&p.scale[col]);
    uint32_t raw[(CAND_CAP + 31) / 32];
#pragma unroll
    for (int t = 0; t < (CAND_CAP + 31) / 32; ++t) {
        const int i = t * 32 + lane;
        raw[t] = 0u;
        if (i < (int)n) {
            const size_t at = (size_t)col * CAND_CAP + i;
            const uint32_t row = DASS_LD(&p.cand.idx[at]);
            raw[t] = DASS_LD(&p.cand.raw[at]);
            const float s = p.scale_per_row ? DASS_LD_G(p.scale + row) : col_scale;
            cand[w].key[i] = DASS_LD(&p.cand.key[at]);
            cand[w].idx[i] = row;
            cand[w].k64[i] = exact_key(fabsf(__uint_as_float(raw[t])), s);
        }
    }
    if (lane == 0) { fl[w].ncoll = n; fl[w].bucket = bucket; fl[w].krem2 = (uint32_t)(r.tau64 >> 32); fl[w].ok = 1u; }
    __syncwarp();
    bracket_rank(cand[w], fl[w], lane);
    __syncwarp();
    if (!fl[w].ok) {
        if (lane == 0) atomicMax(p.status, (int)DASS_ERR_INTERNAL);
        return;
    }
    const LineResult res = fl[w].res;
#pragma unroll
    for (int t = 0; t < (CAND_CAP + 31) / 32; ++t) {
        const int i = t * 32 + lane;
        if (i < (int)n) {
            const uint32_t key = cand[w].key[i], row = cand[w].idx[i];
            const unsigned long long k64 = cand[w].k64[i];
            const bool stays = key > res.tau32 ||
                               (key == res.tau32 && (!res.exact || k64 > res.tau64 || (k64 == res.tau64 && (long long)row <= res.cut)));
            if (stays) {
                if (p.mask) atomicOr(p.mask + (int64_t)row * p.wpr + (col >> 5), 1u << (col & 31));
                if (p.Wp) DASS_ST(p.Wp + (int64_t)row * p.ld + col, (uint16_t)(raw[t] >> 16));
            }
        }
    }
    if (lane == 0) DASS_ST(&p.results[col], res);    // the column's completed rule
}

static cudaError_t launch_emit_stream(const void *W, void *Wp, uint32_t *mask, const float *scale, LineResult *results,
                                      const CandLists &cand, int64_t rows, int64_t cols, int64_t ld, int scale_per_row,
                                      cudaStream_t st)
{
    EmitStreamParams p;
    p.W = static_cast<const uint16_t *>(W);
    p.Wp = static_cast<uint16_t *>(Wp);
    p.mask = mask; p.scale = scale; p.results = results; p.cand = cand;
    p.ld = ld; p.wpr = (cols + 31) / 32;
    p.scale_per_row = scale_per_row;
    CUtensorMap map;
    int64_t grid = 0;
    cudaError_t e = unit_grid_setup(p, &map, &grid, W, rows, cols, ld, true);
    if (e != cudaSuccess) return e;
    static DeviceMask configured{0ull};
    static DeviceMask configured_col{0ull};
    e = scale_per_row ? ensure_dynamic_smem(select_emit_stream_kernel<true>, (int)pn_smem_bytes(SE_STAGES), configured)
                      : ensure_dynamic_smem(select_emit_stream_kernel<false>, (int)pn_smem_bytes(SE_STAGES), configured_col);
    if (e != cudaSuccess) return e;
    if (scale_per_row) select_emit_stream_kernel<true><<<(unsigned)grid, PN_THREADS, pn_smem_bytes(SE_STAGES), st>>>(map, p);
    else select_emit_stream_kernel<false><<<(unsigned)grid, PN_THREADS, pn_smem_bytes(SE_STAGES), st>>>(map, p);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    FixParams f;
    f.results = results; f.cand = cand; f.scale = scale;
    f.Wp = static_cast<uint16_t *>(Wp); f.mask = mask;
    f.cols = cols; f.ld = ld; f.wpr = p.wpr;
    f.scale_per_row = scale_per_row;
    f.status = p.status;
    select_fix_cols_kernel<<<(unsigned)((cols + FIX_WARPS - 1) / FIX_WARPS), FIX_WARPS * 32, 0, st>>>(f);
    return cudaGetLastError();
}

cudaError_t select_launch_emit(const SelectParams &p, bool bf16, const CandLists &cand, int scale_per_row, cudaStream_t st)
{
    if (bf16)   // the TMA-fed streaming pass, then the ranking of the undecided bins
        return launch_emit_stream(p.W, p.Wp, p.mask, p.scale, p.results, cand, p.rows, p.cols, p.ld, scale_per_row, st);
    EmitParams q;
    q.W = p.W; q.Wp = p.Wp; q.mask = p.mask; q.scale = p.scale; q.results = p.results;
    q.rows = p.rows; q.cols = p.cols; q.ld = p.ld; q.wpr = p.wpr;
    q.col_blocks = (p.cols + 255) / 256;
    q.row_blocks = (p.rows + 31) / 32;
    q.scale_per_row = scale_per_row;
    const int64_t want = (q.col_blocks * q.row_blocks + 7) / 8;
    const int64_t cap = (int64_t)device_sm_count() * 8;
    select_emit_cols_kernel<false><<<(int)(want < cap ? want : cap), 256, 0, st>>>(q);
    return cudaGetLastError();
}

}  // namespace dass
