// Stage (b), compression of bf16 weights whose groups run along the columns (the down projection):
// survivors are compacted with byte permutes driven by a shared-memory table instead of per-element
// select chains.
//
// A lane holds 8 consecutive bf16 (16 bytes, four words) of a row and their 8 mask bits.  The table maps
// the mask byte to (a) two permute selectors per output word -- stage 1 picks a 16-bit half out of each
// word pair (x,y) and (z,w), stage 2 picks between the two results -- and (b) the metadata byte.  So a
// compacted output word costs one table load and three permutes whatever the n:m pattern is.
#include "dass_device.cuh"

namespace dass {

struct CompressFastParams {
    const uint16_t *W;
    const uint32_t *mask;
    uint16_t *values;
    uint32_t *meta;
    int64_t rows, cols, ld;
    int64_t wpr, vcols, mwpl;
    int n_keep, m, log2m;
    int two_four;
    int vec_ok;
};

constexpr int CF_THREADS = 256;
constexpr int CF_COLS = 256;

__device__ __forceinline__ uint32_t prmt_c(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// Table entry for (mask byte, output word w): low 16 bits = stage-1 selector, high 16 bits = stage-2
// selector, for the survivors number 2w and 2w+1 (in index order) of the 8 elements.
__device__ __forceinline__ uint32_t make_selectors(uint32_t byte, int w)
{
    int pos[8];
    int n = 0;
    for (int j = 0; j < 8; ++j)
        if ((byte >> j) & 1u) pos[n++] = j;
    for (int k = n; k < 8; ++k) pos[k] = 0;
    const uint32_t pa = (uint32_t)pos[2 * w], pb = (uint32_t)pos[2 * w + 1];
    const uint32_t i = 2u * (pa & 3u), j = 2u * (pb & 3u);           // byte offset inside a word pair
    const uint32_t s1 = (i | ((i + 1u) << 4)) | ((j | ((j + 1u) << 4)) << 8);
    const uint32_t s2 = 0x3210u + (pa >> 2) * 0x0044u + (pb >> 2) * 0x4400u;
    return s1 | (s2 << 16);
}

// 2:4 metadata byte of a mask byte: per 4-bit group pos_lo | pos_hi << 2 (0 for a group without two bits).
__device__ __forceinline__ uint32_t make_meta_2of4(uint32_t byte)
{
    uint32_t out = 0;
    for (int g = 0; g < 2; ++g) {
        const uint32_t nib = (byte >> (4 * g)) & 0xfu;
        const uint32_t lo = nib ? (uint32_t)(__ffs(nib) - 1) : 0u;
        const uint32_t hi = nib ? (uint32_t)(31 - __clz(nib)) : 0u;
        out |= (lo | (hi << 2)) << (4 * g);
    }
    return out;
}

// A warp task is 8 rows x 256 columns: a lane issues the loads of its 8 rows (and their mask words) back to back
// and then works through them, so 16 independent requests per lane are in flight (measured faster than a
// cp.async slab ring of 4-row units: 151 against 170 us on the 70B-shaped down projection).
constexpr int CD_ROWS = 8;

__global__ void __launch_bounds__(CF_THREADS, 3) compress_cols_bf16_kernel(const CompressFastParams p)
{
    __shared__ uint32_t sel_lut[4][256];
    __shared__ uint8_t meta_lut[256];
    for (int e = threadIdx.x; e < 1024; e += CF_THREADS) sel_lut[e >> 8][e & 255] = make_selectors(e & 255, e >> 8);
    if (threadIdx.x < 256) meta_lut[threadIdx.x] = (uint8_t)(p.two_four ? make_meta_2of4(threadIdx.x) : threadIdx.x);
    __syncthreads();

    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (CF_THREADS / 32) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (CF_THREADS / 32);
    const int64_t strips = (p.cols + CF_COLS - 1) / CF_COLS;
    const int64_t row_blocks = (p.rows + CD_ROWS - 1) / CD_ROWS;
    const int64_t ntasks = strips * row_blocks;

    for (int64_t task = warp; task < ntasks; task += nwarps) {
        const int64_t strip = task % strips, rb = task / strips;
        const int64_t r0 = rb * CD_ROWS;
        const int64_t c0 = strip * CF_COLS + lane * 8;
        const int64_t left = p.cols - c0;
        const int nvalid = left >= 8 ? 8 : (left > 0 ? (int)left : 0);     // a multiple of m
        const int nout = (nvalid >> p.log2m) * p.n_keep;
        uint4 v[CD_ROWS];
        uint32_t mw[CD_ROWS];
#pragma unroll
        for (int i = 0; i < CD_ROWS; ++i) {
            const bool ok = nvalid > 0 && r0 + i < p.rows;
            // the row pitch is a multiple of 8 elements: a whole vector stays inside the row's pitch
            v[i] = ok ? DASS_LD_CS(reinterpret_cast<const uint4 *>(p.W + (r0 + i) * p.ld + c0)) : make_uint4(0u, 0u, 0u, 0u);
            mw[i] = ok ? DASS_LD_G(p.mask + (r0 + i) * p.wpr + (c0 >> 5)) : 0u;
        }
        uint16_t *dst = p.values + r0 * p.vcols + (c0 >> p.log2m) * p.n_keep;
        uint32_t *mdst = p.meta + r0 * p.mwpl + (c0 >> 5);
        // whole tiles of a half-density pattern (2:4, 4:8: four survivors per lane and row, one 8-byte store):
        // the common case, decided once per task for the whole warp
        const bool whole = p.vec_ok && nout == 4 && r0 + CD_ROWS <= p.rows &&
                           (strip + 1) * CF_COLS <= p.cols;
        if (whole) {
#pragma unroll
            for (int i = 0; i < CD_ROWS; ++i, dst += p.vcols, mdst += p.mwpl) {
                const uint32_t mb = (mw[i] >> (8 * (lane & 3))) & 0xffu;
                const uint32_t word = quad_pack_bytes((uint32_t)meta_lut[mb], lane);
                if ((lane & 3) == 0) DASS_ST(mdst, word);
                const uint32_t s0 = sel_lut[0][mb], s1 = sel_lut[1][mb];
                const uint32_t o0 = prmt_c(prmt_c(v[i].x, v[i].y, s0 & 0xffffu), prmt_c(v[i].z, v[i].w, s0 & 0xffffu), s0 >> 16);
                const uint32_t o1 = prmt_c(prmt_c(v[i].x, v[i].y, s1 & 0xffffu), prmt_c(v[i].z, v[i].w, s1 & 0xffffu), s1 >> 16);
                DASS_ST_CS(reinterpret_cast<uint2 *>(dst), make_uint2(o0, o1));
            }
            continue;
        }
#pragma unroll
        for (int i = 0; i < CD_ROWS; ++i, dst += p.vcols, mdst += p.mwpl) {
            const uint32_t mb = (mw[i] >> (8 * (lane & 3))) & 0xffu;
            const uint32_t word = quad_pack_bytes((uint32_t)meta_lut[mb], lane);
            if (nvalid == 0 || r0 + i >= p.rows) continue;
            if ((lane & 3) == 0) DASS_ST(mdst, word);
            uint32_t out[4];
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                if (2 * w < nout) {
                    const uint32_t s = sel_lut[w][mb];
                    const uint32_t t_lo = prmt_c(v[i].x, v[i].y, s & 0xffffu);
                    const uint32_t t_hi = prmt_c(v[i].z, v[i].w, s & 0xffffu);
                    out[w] = prmt_c(t_lo, t_hi, s >> 16);
                } else {
                    out[w] = 0u;
                }
            }
            if (nout == 4 && p.vec_ok) {
                DASS_ST_CS(reinterpret_cast<uint2 *>(dst), make_uint2(out[0], out[1]));
            } else {
                for (int k = 0; k < nout; ++k) {
                    const uint32_t ow = k < 2 ? out[0] : k < 4 ? out[1] : k < 6 ? out[2] : out[3];
                    DASS_ST(&dst[k], (uint16_t)((k & 1) ? (ow >> 16) : (ow & 0xffffu)));
                }
            }
        }
    }
}

int device_sm_count();   // dass_abi.cu

cudaError_t compress_cols_bf16_launch(const void *W, const uint32_t *mask_bits, int64_t rows, int64_t cols, int64_t ld,
                                      int n_keep, int m, void *values, uint32_t *meta, cudaStream_t st)
{
    CompressFastParams p;
    p.W = static_cast<const uint16_t *>(W);
    p.mask = mask_bits;
    p.values = static_cast<uint16_t *>(values);
    p.meta = meta;
    p.rows = rows; p.cols = cols; p.ld = ld;
    p.wpr = (cols + 31) / 32;
    p.vcols = cols / m * n_keep;
    p.mwpl = (cols + 31) / 32;             // 4-bit fields per 4 columns or m-bit fields per m columns: one bit per column
    p.n_keep = n_keep; p.m = m; p.log2m = m == 8 ? 3 : 2;
    p.two_four = (n_keep == 2 && m == 4) ? 1 : 0;
    p.vec_ok = ((p.vcols * 2) % 16 == 0) && ((reinterpret_cast<uintptr_t>(values) & 15u) == 0);
    const int64_t strips = (cols + CF_COLS - 1) / CF_COLS;
    const int64_t tasks = strips * ((rows + CD_ROWS - 1) / CD_ROWS);
    const int64_t wpb = CF_THREADS / 32;
    const int64_t want = (tasks + wpb - 1) / wpb;
    const int64_t cap = (int64_t)device_sm_count() * 8;
    const int grid = (int)(want < cap ? want : cap);
    compress_cols_bf16_kernel<<<grid, CF_THREADS, 0, st>>>(p);
    return cudaGetLastError();
}

}  // namespace dass
