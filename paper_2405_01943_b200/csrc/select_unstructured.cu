// Unstructured DaSS selection at a sparsity ratio s (Section 3, "Pruning Granularity"): in every comparison
// line -- a column of Wg / Wu (all neurons at one input: input-balanced) or a row of Wd (output-balanced) --
// the floor(s * L) weights with the lowest Eq. 4 / Eq. 5 score are pruned.  No sort: an exact radix select.
//
// A CTA caches its lines (two of them) in shared memory and finds, per line, the k-th largest 64-bit key in
// eight 8-bit passes; the key is the bit pattern of the exact double product |w| * scale, which orders like the
// real score.  A last pass keeps every key above the threshold and, among keys equal to it, the ones with the
// lowest indices (found with an ordered prefix count), which is the oracle's "higher score first, lower index
// first" order.  Lines that are matrix rows are read with 16-byte loads; lines that are matrix columns are read
// two adjacent columns at a time (4 or 8 bytes per row, neighbouring CTAs share the sectors through L2) and
// their mask bits are OR-ed into the packed mask with atomics (the mask is zeroed first).
#include <cmath>
#include <type_traits>

#include "dass_device.cuh"

namespace dass {

constexpr int U_THREADS = 256;
constexpr int U_LINES = 2;            // lines per CTA
constexpr int U_WARPS = U_THREADS / 32;

struct SelectParams {
    const void *W;
    void *Wp;            // nullable
    uint32_t *mask;      // nullable
    const float *scale;  // precomputed fl32(norm^alpha)
    int64_t rows, cols, ld;
    int64_t wpr;
    int64_t L;           // line length
    int64_t nlines;
    int64_t lpad;        // L rounded up to 8
    uint32_t k;          // survivors per line
    int scale_along_line;   // 1: scale[e] varies along the line; 0: scale[line]
};

__global__ void scale_vector_kernel(const float *__restrict__ norm, int64_t n, int mode, float alpha, float *__restrict__ out)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = scale_from_norm(norm[i], mode, alpha);
}

template <bool BF16>
__device__ __forceinline__ double key_of(uint32_t raw, float scale)
{
    const float a = BF16 ? __uint_as_float((raw & 0x7fffu) << 16) : __uint_as_float(raw & 0x7fffffffu);
    return (double)a * (double)scale;     // exact: at most 24 + 24 significant bits
}

// LINE_IS_ROW: the CTA's two lines are matrix rows 2b, 2b+1 (threads 0..127 work on the first, 128..255 on
// the second).  Otherwise they are the matrix columns 2b, 2b+1 and every thread works on both.
template <bool BF16, bool LINE_IS_ROW>
__global__ void __launch_bounds__(U_THREADS) select_unstructured_kernel(const SelectParams p)
{
    using elem_t = typename std::conditional<BF16, uint16_t, uint32_t>::type;
    extern __shared__ __align__(16) unsigned char u_smem[];
    elem_t *line_mem = reinterpret_cast<elem_t *>(u_smem);                       // [U_LINES][lpad]
    uint32_t *hist = reinterpret_cast<uint32_t *>(u_smem + (size_t)U_LINES * p.lpad * sizeof(elem_t));   // [U_LINES][U_WARPS][256]
    __shared__ unsigned long long s_prefix[U_LINES];
    __shared__ uint32_t s_krem[U_LINES];
    __shared__ uint32_t s_warp_tot[U_WARPS];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t line0 = (int64_t)blockIdx.x * U_LINES;
    const int nl = (int)((p.nlines - line0) < U_LINES ? (p.nlines - line0) : U_LINES);
    const int64_t nchunks = p.lpad >> 3;
    constexpr int TPL = LINE_IS_ROW ? U_THREADS / U_LINES : U_THREADS;          // threads per line
    const int my_first = LINE_IS_ROW ? tid / TPL : 0;                           // first line this thread works on
    const int my_count = LINE_IS_ROW ? 1 : U_LINES;
    const int tau = LINE_IS_ROW ? tid % TPL : tid;                              // index among the line's threads

    // ---------------------------------------------------------------- phase 0: lines -> shared memory
    if constexpr (LINE_IS_ROW) {
        const int ln = my_first;
        if (ln < nl) {
            const elem_t *src = static_cast<const elem_t *>(p.W) + (line0 + ln) * p.ld;
            for (int64_t e = tau; e < p.lpad; e += TPL) line_mem[ln * p.lpad + e] = e < p.L ? src[e] : (elem_t)0;
        }
    } else {
        const elem_t *src = static_cast<const elem_t *>(p.W) + line0;            // column line0 of row r at src[r * ld]
        for (int64_t r = tid; r < p.lpad; r += U_THREADS) {
#pragma unroll
            for (int ln = 0; ln < U_LINES; ++ln)
                line_mem[ln * p.lpad + r] = (r < p.L && ln < nl) ? src[r * p.ld + ln] : (elem_t)0;
        }
    }
    if (tid < U_LINES) { s_prefix[tid] = 0ull; s_krem[tid] = p.k; }
    __syncthreads();

    // ---------------------------------------------------------------- phase 1: radix select, 8 bits per pass
    for (int shift = 56; shift >= 0; shift -= 8) {
        for (int i = tid; i < U_LINES * U_WARPS * 256; i += U_THREADS) hist[i] = 0u;
        __syncthreads();
        const unsigned long long known = shift == 56 ? 0ull : (~0ull << (shift + 8));
        for (int m = 0; m < my_count; ++m) {
            const int ln = my_first + m;
            if (ln >= nl) continue;
            const unsigned long long prefix = s_prefix[ln];
            const float line_scale = p.scale_along_line ? 0.0f : p.scale[line0 + ln];
            uint32_t *h = hist + (ln * U_WARPS + warp) * 256;
            for (int64_t q = tau; q < nchunks; q += TPL) {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int64_t e = q * 8 + j;
                    if (e < p.L) {
                        const float sc = p.scale_along_line ? __ldg(p.scale + e) : line_scale;
                        const unsigned long long key = (unsigned long long)__double_as_longlong(key_of<BF16>(line_mem[ln * p.lpad + e], sc));
                        if (((key ^ prefix) & known) == 0ull) atomicAdd(h + (uint32_t)((key >> shift) & 0xffull), 1u);
                    }
                }
            }
        }
        __syncthreads();
        // one warp per line finds the bucket that holds the k_rem-th largest candidate
        if (warp < nl) {
            const int ln = warp;
            uint32_t cnt[8], lane_sum = 0u;
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                uint32_t c = 0u;
                for (int w = 0; w < U_WARPS; ++w) c += hist[(ln * U_WARPS + w) * 256 + lane * 8 + b];
                cnt[b] = c;
                lane_sum += c;
            }
            uint32_t v = lane_sum;                          // becomes the sum over lanes >= this one
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t t = __shfl_down_sync(FULL_MASK, v, off);
                if (lane + off < 32) v += t;
            }
            uint32_t above = v - lane_sum;                  // candidates in higher buckets than this lane's
            const uint32_t krem = s_krem[ln];
            const bool mine = above < krem && krem <= above + lane_sum;
            uint32_t digit = 0u, greater = 0u;
            if (mine) {
#pragma unroll
                for (int b = 7; b >= 0; --b) {
                    if (krem <= above + cnt[b]) { digit = (uint32_t)(lane * 8 + b); greater = above; break; }
                    above += cnt[b];
                }
            }
            const uint32_t who = __ballot_sync(FULL_MASK, mine);
            const int src = who ? __ffs(who) - 1 : 0;
            digit = __shfl_sync(FULL_MASK, digit, src);
            greater = __shfl_sync(FULL_MASK, greater, src);
            if (lane == 0) {
                s_prefix[ln] |= (unsigned long long)digit << shift;
                s_krem[ln] = krem - greater;
            }
        }
        __syncthreads();
    }

    // ---------------------------------------------------------------- phase 2: emit in index order
    const int64_t nbatches = (nchunks + TPL - 1) / TPL;
    for (int m = 0; m < my_count; ++m) {
        const int ln = my_first + m;
        const bool live = ln < nl;
        const unsigned long long tau_key = live ? s_prefix[ln] : 0ull;
        const uint32_t need = live ? s_krem[ln] : 0u;       // how many of the keys equal to the threshold stay
        const float line_scale = (!live || p.scale_along_line) ? 0.0f : p.scale[line0 + ln];
        uint32_t base = 0u;                                  // equal keys seen before this batch
        for (int64_t bt = 0; bt < nbatches; ++bt) {
            const int64_t q = bt * TPL + tau;
            uint32_t gt = 0u, eq = 0u;
            if (live && q < nchunks) {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int64_t e = q * 8 + j;
                    if (e < p.L) {
                        const float sc = p.scale_along_line ? __ldg(p.scale + e) : line_scale;
                        const unsigned long long key = (unsigned long long)__double_as_longlong(key_of<BF16>(line_mem[ln * p.lpad + e], sc));
                        gt |= (key > tau_key ? 1u : 0u) << j;
                        eq |= (key == tau_key ? 1u : 0u) << j;
                    }
                }
            }
            // exclusive prefix of the equal counts over the line's threads, in thread (= index) order
            const uint32_t mycnt = __popc(eq);
            uint32_t incl = mycnt;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t t = __shfl_up_sync(FULL_MASK, incl, off);
                if (lane >= off) incl += t;
            }
            if (lane == 31) s_warp_tot[warp] = incl;
            __syncthreads();
            const int w_first = LINE_IS_ROW ? (tid / TPL) * (TPL / 32) : 0;     // first warp of this line
            uint32_t before = base, batch_total = 0u;
            for (int w = 0; w < TPL / 32; ++w) {
                const uint32_t t = s_warp_tot[w_first + w];
                if (w_first + w < warp) before += t;
                batch_total += t;
            }
            __syncthreads();
            uint32_t rank = before + incl - mycnt;           // equal keys with a lower index than this thread's first
            uint32_t keep = gt;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if ((eq >> j) & 1u) {
                    if (rank < need) keep |= 1u << j;
                    ++rank;
                }
            }
            base += batch_total;

            if (live && q < nchunks) {
                const int64_t e0 = q * 8;
                const int64_t left = p.L - e0;
                const int nvalid = left >= 8 ? 8 : (int)left;
                if constexpr (LINE_IS_ROW) {
                    const int64_t r = line0 + ln;
                    // consecutive threads hold consecutive 8-column chunks: four of them make a mask word
                    if (p.mask) {
                        uint8_t *mrow = reinterpret_cast<uint8_t *>(p.mask + r * p.wpr);
                        mrow[q] = (uint8_t)keep;             // byte q = columns 8q..8q+7 (little endian words)
                    }
                    if (p.Wp) {
                        elem_t *dst = static_cast<elem_t *>(p.Wp) + r * p.ld + e0;
                        const elem_t *srcl = line_mem + ln * p.lpad + e0;
                        if (nvalid == 8) {      // whole chunk: 16-byte stores (rows are 16-byte aligned by the ld rule)
                            constexpr int EPV = 16 / sizeof(elem_t);     // elements per vector
#pragma unroll
                            for (int vsel = 0; vsel < 8 / EPV; ++vsel) {
                                uint4 x = reinterpret_cast<const uint4 *>(srcl)[vsel];
                                uint32_t *xw = reinterpret_cast<uint32_t *>(&x);
#pragma unroll
                                for (int wi = 0; wi < 4; ++wi) {
                                    if constexpr (BF16) {
                                        const uint32_t mm = (keep >> (2 * wi)) & 3u;
                                        xw[wi] &= ((mm & 1u) ? 0x0000ffffu : 0u) | ((mm & 2u) ? 0xffff0000u : 0u);
                                    } else {
                                        xw[wi] = ((keep >> (vsel * 4 + wi)) & 1u) ? xw[wi] : 0u;
                                    }
                                }
                                reinterpret_cast<uint4 *>(dst)[vsel] = x;
                            }
                        } else {
                            for (int j = 0; j < nvalid; ++j) dst[j] = ((keep >> j) & 1u) ? srcl[j] : (elem_t)0;
                        }
                    }
                } else {
                    const int64_t c = line0 + ln;
                    for (int j = 0; j < nvalid; ++j) {
                        const int64_t r = e0 + j;
                        const bool kp = (keep >> j) & 1u;
                        if (p.mask && kp) atomicOr(p.mask + r * p.wpr + (c >> 5), 1u << (c & 31));
                        if (p.Wp) static_cast<elem_t *>(p.Wp)[r * p.ld + c] = kp ? line_mem[ln * p.lpad + r] : (elem_t)0;
                    }
                }
            }
        }
    }
}

size_t select_smem_bytes(int64_t L, bool bf16)
{
    const int64_t lpad = (L + 7) / 8 * 8;
    return (size_t)U_LINES * lpad * (bf16 ? 2 : 4) + (size_t)U_LINES * U_WARPS * 256 * sizeof(uint32_t);
}

template <bool BF16, bool ROW>
static cudaError_t launch_select(const SelectParams &p, size_t smem, cudaStream_t st)
{
    cudaError_t e = cudaFuncSetAttribute(select_unstructured_kernel<BF16, ROW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int64_t grid = (p.nlines + U_LINES - 1) / U_LINES;
    select_unstructured_kernel<BF16, ROW><<<(unsigned)grid, U_THREADS, smem, st>>>(p);
    return cudaGetLastError();
}

cudaError_t select_unstructured_launch(const void *W, int64_t rows, int64_t cols, int64_t ld, bool bf16,
                                       const float *norm, bool norm_cols, float alpha, uint32_t k, bool line_is_row,
                                       uint32_t *mask_bits, void *W_pruned, float *scale_ws, cudaStream_t st)
{
    const int64_t n_norm = norm_cols ? cols : rows;
    scale_vector_kernel<<<(unsigned)((n_norm + 255) / 256), 256, 0, st>>>(norm, n_norm, (int)scale_mode_for(alpha), alpha, scale_ws);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    SelectParams p;
    p.W = W; p.Wp = W_pruned; p.mask = mask_bits; p.scale = scale_ws;
    p.rows = rows; p.cols = cols; p.ld = ld;
    p.wpr = (cols + 31) / 32;
    p.L = line_is_row ? cols : rows;
    p.nlines = line_is_row ? rows : cols;
    p.lpad = (p.L + 7) / 8 * 8;
    p.k = k;
    p.scale_along_line = (line_is_row == norm_cols) ? 1 : 0;   // the norm index runs along the line
    if (mask_bits) {
        // column lines OR their bits in; row lines write whole bytes but leave the row padding untouched
        e = cudaMemsetAsync(mask_bits, 0, (size_t)rows * p.wpr * sizeof(uint32_t), st);
        if (e != cudaSuccess) return e;
    }
    const size_t smem = select_smem_bytes(p.L, bf16);
    if (bf16) return line_is_row ? launch_select<true, true>(p, smem, st) : launch_select<true, false>(p, smem, st);
    return line_is_row ? launch_select<false, true>(p, smem, st) : launch_select<false, false>(p, smem, st);
}

}  // namespace dass

using namespace dass;

extern "C" dass_status dass_select_workspace_bytes(int64_t rows, int64_t cols, dass_axis norm_axis, size_t *bytes)
{
    if (!bytes) return DASS_ERR_NULL;
    if (norm_axis != DASS_AXIS_ROWS && norm_axis != DASS_AXIS_COLS) return DASS_ERR_DTYPE;
    if (rows < 1 || cols < 1) return DASS_ERR_SHAPE;
    *bytes = (size_t)(norm_axis == DASS_AXIS_ROWS ? rows : cols) * sizeof(float);
    return DASS_OK;
}

extern "C" dass_status dass_select_unstructured(const void *W, int64_t rows, int64_t cols, int64_t ld, dass_dtype dt,
                                                const float *norm, dass_axis norm_axis, float alpha,
                                                double sparsity, dass_axis compare_axis,
                                                uint32_t *mask_bits, void *W_pruned,
                                                void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!W || !norm || (!mask_bits && !W_pruned)) return DASS_ERR_NULL;
    if (dt != DASS_BF16 && dt != DASS_F32) return DASS_ERR_DTYPE;
    if ((norm_axis != DASS_AXIS_ROWS && norm_axis != DASS_AXIS_COLS) ||
        (compare_axis != DASS_AXIS_ROWS && compare_axis != DASS_AXIS_COLS)) return DASS_ERR_DTYPE;
    if (rows < 1 || cols < 1 || ld < cols) return DASS_ERR_SHAPE;
    if (!(sparsity >= 0.0 && sparsity < 1.0)) return DASS_ERR_SHAPE;
    if (!std::isfinite(alpha) || alpha < 0.0f) return DASS_ERR_UNSUPPORTED;
    const bool bf16 = dt == DASS_BF16;
    if (ld % (bf16 ? 8 : 4) != 0) return DASS_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(W) & 15u) || (W_pruned && (reinterpret_cast<uintptr_t>(W_pruned) & 15u)) ||
        (reinterpret_cast<uintptr_t>(norm) & 3u) || (reinterpret_cast<uintptr_t>(mask_bits) & 3u)) return DASS_ERR_ALIGN;
    size_t need = 0;
    const dass_status qs = dass_select_workspace_bytes(rows, cols, norm_axis, &need);
    if (qs != DASS_OK) return qs;
    if (!workspace || workspace_bytes < need) return DASS_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 15u) return DASS_ERR_ALIGN;
    const bool line_is_row = compare_axis == DASS_AXIS_COLS;         // the index that varies inside a line
    const int64_t L = line_is_row ? cols : rows;
    if (L >= (int64_t)1 << 31) return DASS_ERR_UNSUPPORTED;
    if (select_smem_bytes(L, bf16) > (size_t)220 * 1024) return DASS_ERR_UNSUPPORTED;   // two lines must fit in shared memory
    const int64_t n_prune = (int64_t)std::floor(sparsity * (double)L);
    const uint32_t k = (uint32_t)(L - n_prune);
    if (select_unstructured_launch(W, rows, cols, ld, bf16, norm, norm_axis == DASS_AXIS_COLS, alpha, k, line_is_row,
                                   mask_bits, W_pruned, static_cast<float *>(workspace),
                                   static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return DASS_ERR_CUDA;
    return DASS_OK;
}
