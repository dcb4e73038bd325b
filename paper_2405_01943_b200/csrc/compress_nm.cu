// Stage (b), last step: N:M compressed values + metadata from the weights and the packed mask.
//
// Same tiling as the scoring pass (a warp owns 32 rows x 256 columns, a lane 8 consecutive columns),
// so weight loads and value stores stay 128-bit and coalesced for either group axis.  Metadata
// fields are produced in registers and packed into 32-bit words with warp shuffles (groups along the
// columns: four lanes share a word) or directly per lane (groups along the rows: a lane's 8 columns
// fill whole words).  Bandwidth-bound: reads W and one mask bit per weight, writes n_keep/m of W plus
// the fields.  These generic kernels serve fp32 weights and bf16 row groups (2:4 and 4:8 row groups have a kernel
// of their own below); bf16 column groups take the permute-table kernel of compress_nm_bf16.cu.
#include "dass_device.cuh"
#include "nm_compact.cuh"

namespace dass {

struct CompressParams {
    const void *W;
    const uint32_t *mask;
    void *values;
    uint32_t *meta;
    int64_t rows, cols, ld;
    int64_t wpr;          // mask words per row
    int64_t vcols;        // columns of the values matrix
    int64_t mwpl;         // metadata words per line
    int64_t col_blocks, row_blocks;
    int n_keep;
    int vec_ok;           // values rows are 16-byte aligned: vector stores allowed
};

constexpr int C_TILE_ROWS = 32;
constexpr int C_TILE_COLS = 256;
constexpr int C_THREADS = 256;

// ---------------------------------------------------------------- groups along the columns
template <bool BF16, int M, bool TWO_FOUR>
__global__ void __launch_bounds__(C_THREADS) compress_group_cols_kernel(const CompressParams p)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (C_THREADS / 32) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (C_THREADS / 32);
    const int64_t ntasks = p.col_blocks * p.row_blocks;
    constexpr int UNROLL = 4;

    for (int64_t task = warp; task < ntasks; task += nwarps) {
        const int64_t cb = task % p.col_blocks;
        const int64_t rb = task / p.col_blocks;
        const int64_t c0 = cb * C_TILE_COLS + lane * 8;
        const int64_t left = p.cols - c0;
        const int nvalid = left >= 8 ? 8 : (left > 0 ? (int)left : 0);   // a multiple of M
        const int nout = nvalid / M * p.n_keep;                           // values this lane emits per row

        for (int i = 0; i < C_TILE_ROWS; i += UNROLL) {
            const int64_t rbase = rb * C_TILE_ROWS + i;
            if (rbase >= p.rows) break;
            Chunk<BF16> ch[UNROLL];
            uint32_t mbyte[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                if (rbase + u < p.rows && nvalid > 0) {
                    chunk_load<BF16>(ch[u], p.W, (rbase + u) * p.ld + c0, nvalid);
                    mbyte[u] = (DASS_LD_G(p.mask + (rbase + u) * p.wpr + (c0 >> 5)) >> (8 * (lane & 3))) & 0xffu;
                } else {
                    chunk_zero<BF16>(ch[u]);
                    mbyte[u] = 0u;
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int64_t r = rbase + u;
                Chunk<BF16> out;
                const uint32_t field_byte = compact_cols<BF16, M, TWO_FOUR>(ch[u], mbyte[u], p.n_keep, nout, out);
                const uint32_t word = quad_pack_bytes(field_byte, lane);
                if (r < p.rows && nvalid > 0) {
                    if ((lane & 3) == 0) DASS_ST(&p.meta[r * p.mwpl + (c0 >> 5)], word);
                    chunk_store_n<BF16>(out, p.values, r * p.vcols + c0 / M * p.n_keep, nout, p.vec_ok != 0);
                }
            }
        }
    }
}

// ---------------------------------------------------------------- groups along the rows
template <bool BF16, int M, bool TWO_FOUR>
__global__ void __launch_bounds__(C_THREADS) compress_group_rows_kernel(const CompressParams p)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (C_THREADS / 32) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (C_THREADS / 32);
    const int64_t ntasks = p.col_blocks * p.row_blocks;
    constexpr int MAXK = TWO_FOUR ? 2 : M - 1;   // survivors per group that can occur

    for (int64_t task = warp; task < ntasks; task += nwarps) {
        const int64_t cb = task % p.col_blocks;
        const int64_t rb = task / p.col_blocks;
        const int64_t c0 = cb * C_TILE_COLS + lane * 8;
        const int64_t left = p.cols - c0;
        const int nvalid = left >= 8 ? 8 : (left > 0 ? (int)left : 0);
        if (nvalid == 0) continue;   // no shuffles in this kernel: lanes are independent

        for (int g = 0; g < C_TILE_ROWS / M; ++g) {
            const int64_t r0 = rb * C_TILE_ROWS + g * M;
            if (r0 >= p.rows) break;
            const int64_t line = r0 / M;
            Chunk<BF16> ch[M];
            uint32_t mbyte[M];
#pragma unroll
            for (int q = 0; q < M; ++q) {
                chunk_load<BF16>(ch[q], p.W, (r0 + q) * p.ld + c0, nvalid);
                mbyte[q] = (DASS_LD_G(p.mask + (r0 + q) * p.wpr + (c0 >> 5)) >> (8 * (lane & 3))) & 0xffu;
            }
            Chunk<BF16> out[MAXK];
            uint32_t fields_lo, fields_hi;   // packed fields of columns 0..3 / 4..7 (or all 8 in lo)
            compact_rows<BF16, M, TWO_FOUR, MAXK>(ch, mbyte, p.n_keep, out, fields_lo, fields_hi);
            if constexpr (TWO_FOUR || M == 4) {
                DASS_ST(&p.meta[line * p.mwpl + (c0 >> 3)], fields_lo);
            } else {
                DASS_ST(&p.meta[line * p.mwpl + (c0 >> 2)], fields_lo);
                if (nvalid > 4) DASS_ST(&p.meta[line * p.mwpl + (c0 >> 2) + 1], fields_hi);
            }
#pragma unroll
            for (int k = 0; k < MAXK; ++k)
                if (k < p.n_keep)
                    chunk_store_n<BF16>(out[k], p.values, (line * p.n_keep + k) * p.vcols + c0, nvalid, p.vec_ok != 0);
        }
    }
}

// ---------------------------------------------------------------- bf16, groups along the rows, fast path
// A lane holds 8 rows of its 8 columns (four words per row) and the 8 keep bits of every row: one group of 8 per
// column, or two groups of 4.  The survivors of a column keep their row order, so row q of a group goes to output
// row k = (number of kept rows above q), a small count kept bit-sliced over the 8 columns.  For every possible
// (q, k) the byte "kept and count == k" is spread to 16-bit lane masks (one multiply and a sign-replicating byte
// permute per word pair) and the row is ORed into output k under it: no per-element select chains.
// Metadata: the keep mask of every column is the bit transpose of the keep bytes; the 2:4 nibble
// pos_lo | pos_hi << 2 is the transpose of the bit-sliced positions sum_q q * [row q goes to output k].
__device__ __forceinline__ uint32_t prmt_b32(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// nibble made of bit j of each of the four bytes of x (byte a -> bit a)
__device__ __forceinline__ uint32_t gather_bit(uint32_t x, int j)
{
    return (((x >> j) & 0x01010101u) * 0x10204080u) >> 28;
}

template <int M, int K, bool TWO_FOUR>
__global__ void __launch_bounds__(C_THREADS) compress_rows_bf16_kernel(const CompressParams p)
{
    static_assert((M == 8 && !TWO_FOUR) || (M == 4 && (!TWO_FOUR || K == 2)), "groups of 4 or 8 rows");
    constexpr int G = 8 / M;         // groups in the 8 rows a lane takes at a time
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (C_THREADS / 32) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (C_THREADS / 32);
    const int64_t ntasks = p.col_blocks * p.row_blocks;

    for (int64_t task = warp; task < ntasks; task += nwarps) {
        const int64_t cb = task % p.col_blocks;
        const int64_t rb = task / p.col_blocks;
        const int64_t c0 = cb * C_TILE_COLS + lane * 8;
        const int64_t left = p.cols - c0;
        const int nvalid = left >= 8 ? 8 : (left > 0 ? (int)left : 0);
        if (nvalid == 0) continue;   // no shuffles in this kernel: lanes are independent

        for (int it = 0; it < C_TILE_ROWS / 8; ++it) {
            const int64_t rbase = rb * C_TILE_ROWS + it * 8;
            if (rbase >= p.rows) break;
            Chunk<true> ch[8];
            uint32_t mb[8];
            if (M == 8 || rbase + 8 <= p.rows) {     // all 8 rows exist: eight independent loads in flight
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    chunk_load<true>(ch[q], p.W, (rbase + q) * p.ld + c0, nvalid);
                    mb[q] = (DASS_LD_G(p.mask + (rbase + q) * p.wpr + (c0 >> 5)) >> (8 * (lane & 3))) & 0xffu;
                }
            } else {                                 // rows is a multiple of 4 only: the last group of 4 stands alone
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if (q < 4) {
                        chunk_load<true>(ch[q], p.W, (rbase + q) * p.ld + c0, nvalid);
                        mb[q] = (DASS_LD_G(p.mask + (rbase + q) * p.wpr + (c0 >> 5)) >> (8 * (lane & 3))) & 0xffu;
                    } else {
                        chunk_zero<true>(ch[q]);
                        mb[q] = 0u;
                    }
                }
            }
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const int64_t r0 = rbase + g * M;
                if (r0 < p.rows) {
                    const int64_t line = r0 / M;
                    uint32_t out[K][4];
#pragma unroll
                    for (int k = 0; k < K; ++k)
#pragma unroll
                        for (int w = 0; w < 4; ++w) out[k][w] = 0u;
                    uint32_t b0 = 0u, b1 = 0u, b2 = 0u;          // bit-sliced count of kept rows above the current one
                    uint32_t pos[2][2] = {{0u, 0u}, {0u, 0u}};   // 2:4: bit-sliced position bits of the two survivors
#pragma unroll
                    for (int q = 0; q < M; ++q) {
                        const uint32_t m = mb[g * M + q];
#pragma unroll
                        for (int k = 0; k < K; ++k) {
                            if (k <= q && q - k <= M - K) {   // row q can only land in these outputs
                                const uint32_t eq = ((k & 1) ? b0 : ~b0) & ((k & 2) ? b1 : ~b1) & ((k & 4) ? b2 : ~b2);
                                const uint32_t e = eq & m;
                                const uint32_t zlo = (e & 0xfu) * 0x10204080u;    // bit j -> sign bit of byte j
                                const uint32_t zhi = (e >> 4) * 0x10204080u;
                                const Chunk<true> &row = ch[g * M + q];
                                out[k][0] |= row.w[0] & prmt_b32(zlo, 0u, 0x9988u);
                                out[k][1] |= row.w[1] & prmt_b32(zlo, 0u, 0xbbaau);
                                out[k][2] |= row.w[2] & prmt_b32(zhi, 0u, 0x9988u);
                                out[k][3] |= row.w[3] & prmt_b32(zhi, 0u, 0xbbaau);
                                if constexpr (TWO_FOUR) {
                                    if (q & 1) pos[k][0] |= e;
                                    if (q & 2) pos[k][1] |= e;
                                }
                            }
                        }
                        const uint32_t c0b = b0 & m;
                        b0 ^= m;
                        const uint32_t c1b = b1 & c0b;
                        b1 ^= c0b;
                        b2 ^= c1b;
                    }
                    if constexpr (M == 8) {
                        // byte j of (lo, hi) = keep mask of column j (bit q = row q)
                        const uint32_t x = mb[0] | (mb[1] << 8) | (mb[2] << 16) | (mb[3] << 24);
                        const uint32_t y = mb[4] | (mb[5] << 8) | (mb[6] << 16) | (mb[7] << 24);
                        uint32_t fields_lo = 0u, fields_hi = 0u;
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const uint32_t colmask = gather_bit(x, j) | (gather_bit(y, j) << 4);
                            if (j < 4) fields_lo |= colmask << (8 * j);
                            else fields_hi |= colmask << (8 * (j - 4));
                        }
                        DASS_ST(&p.meta[line * p.mwpl + (c0 >> 2)], fields_lo);
                        if (nvalid > 4) DASS_ST(&p.meta[line * p.mwpl + (c0 >> 2) + 1], fields_hi);
                    } else {
                        // nibble j = keep mask of column j, or for 2:4 pos_lo | pos_hi << 2
                        const uint32_t x = TWO_FOUR ? (pos[0][0] | (pos[0][1] << 8) | (pos[1][0] << 16) | (pos[1][1] << 24))
                                                    : (mb[g * M] | (mb[g * M + 1] << 8) | (mb[g * M + 2] << 16) | (mb[g * M + 3] << 24));
                        uint32_t fields = 0u;
#pragma unroll
                        for (int j = 0; j < 8; ++j) fields |= gather_bit(x, j) << (4 * j);
                        DASS_ST(&p.meta[line * p.mwpl + (c0 >> 3)], fields);
                    }
#pragma unroll
                    for (int k = 0; k < K; ++k) {
                        Chunk<true> o;
#pragma unroll
                        for (int w = 0; w < 4; ++w) o.w[w] = out[k][w];
                        chunk_store_n<true>(o, p.values, (line * K + k) * p.vcols + c0, nvalid, p.vec_ok != 0);
                    }
                }
            }
        }
    }
}

template <bool BF16, int M, bool TWO_FOUR>
static cudaError_t launch_compress(const CompressParams &p, bool group_cols, int grid, cudaStream_t st)
{
    if (group_cols) compress_group_cols_kernel<BF16, M, TWO_FOUR><<<grid, C_THREADS, 0, st>>>(p);
    else compress_group_rows_kernel<BF16, M, TWO_FOUR><<<grid, C_THREADS, 0, st>>>(p);
    return cudaGetLastError();
}

int device_sm_count();   // dass_abi.cu
cudaError_t compress_cols_bf16_launch(const void *W, const uint32_t *mask_bits, int64_t rows, int64_t cols, int64_t ld,
                                      int n_keep, int m, void *values, uint32_t *meta, cudaStream_t st);   // compress_nm_bf16.cu

cudaError_t compress_nm_launch(const void *W, const uint32_t *mask_bits, int64_t rows, int64_t cols, int64_t ld,
                               bool bf16, int n_keep, int m, bool group_cols,
                               void *values, uint32_t *meta, cudaStream_t st)
{
    if (bf16 && group_cols)   // permute-table kernel of compress_nm_bf16.cu
        return compress_cols_bf16_launch(W, mask_bits, rows, cols, ld, n_keep, m, values, meta, st);
    CompressParams p;
    p.W = W; p.mask = mask_bits; p.values = values; p.meta = meta;
    p.rows = rows; p.cols = cols; p.ld = ld;
    p.wpr = (cols + 31) / 32;
    const bool two_four = (n_keep == 2 && m == 4);
    const int field_bits = two_four ? 4 : m;
    const int fpw = 32 / field_bits;
    if (group_cols) {
        p.vcols = cols / m * n_keep;
        p.mwpl = (cols / m + fpw - 1) / fpw;
    } else {
        p.vcols = cols;
        p.mwpl = (cols + fpw - 1) / fpw;
    }
    const int esz = bf16 ? 2 : 4;
    p.vec_ok = ((p.vcols * esz) % 16 == 0) && ((reinterpret_cast<uintptr_t>(values) & 15u) == 0);
    p.col_blocks = (cols + C_TILE_COLS - 1) / C_TILE_COLS;
    p.row_blocks = (rows + C_TILE_ROWS - 1) / C_TILE_ROWS;
    p.n_keep = n_keep;
    const int64_t ntasks = p.col_blocks * p.row_blocks;
    const int64_t wpb = C_THREADS / 32;
    const int64_t want = (ntasks + wpb - 1) / wpb;
    const int64_t cap = (int64_t)device_sm_count() * 8;
    const int grid = (int)(want < cap ? want : cap);
    if (bf16) {
        if (!group_cols && m == 8 && n_keep == 4) {      // 4:8 and 2:4 on gate / up: the bit-sliced routing kernel
            compress_rows_bf16_kernel<8, 4, false><<<grid, C_THREADS, 0, st>>>(p);
            return cudaGetLastError();
        }
        if (!group_cols && two_four) {
            compress_rows_bf16_kernel<4, 2, true><<<grid, C_THREADS, 0, st>>>(p);
            return cudaGetLastError();
        }
        if (two_four) return launch_compress<true, 4, true>(p, group_cols, grid, st);
        return m == 4 ? launch_compress<true, 4, false>(p, group_cols, grid, st)
                      : launch_compress<true, 8, false>(p, group_cols, grid, st);
    }
    if (two_four) return launch_compress<false, 4, true>(p, group_cols, grid, st);
    return m == 4 ? launch_compress<false, 4, false>(p, group_cols, grid, st)
                  : launch_compress<false, 8, false>(p, group_cols, grid, st);
}

}  // namespace dass
