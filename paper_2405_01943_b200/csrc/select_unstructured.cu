// Unstructured DaSS selection at a sparsity ratio s (Section 3, "Pruning Granularity"): in every comparison
// line -- a column of Wg / Wu (all neurons at one input: input-balanced) or a row of Wd (output-balanced) --
// the floor(s * L) weights with the lowest Eq. 4 / Eq. 5 score are pruned.  No sort: an exact radix select.
//
// A CTA caches its line(s) in shared memory and finds the threshold in two stages.  Stage A works on the rounded
// products p = fl32(|w| * scale), four 8-bit passes; rounding is monotone, so p decides every pair of weights
// whose rounded products differ.  Only if more products equal the threshold than may stay does stage B repeat the
// selection among those with the exact double products as keys (eight passes); exact ties are then broken towards
// the lower index with an ordered prefix count -- the oracle's "higher score first, lower index first".
// Lines that are matrix rows (one per CTA, 16-byte loads) are emitted by the same kernel.  Lines that are matrix
// columns are read two adjacent columns per CTA (neighbouring CTAs share the 32-byte sectors through L2); the
// kernel publishes (tau32, exact, tau64, cut) per column and select_emit_cols_kernel applies them in a streaming
// pass with coalesced rows.
#include <cmath>
#include <type_traits>

#include "dass_device.cuh"

namespace dass {


// What the selection found for one line; enough to decide every element of the line locally:
// keep iff p > tau32, or p == tau32 and (not exact, or k64 > tau64, or k64 == tau64 and index <= cut).
struct LineResult {
    unsigned long long tau64;
    long long cut;
    uint32_t tau32;
    uint32_t exact;
};

struct SelectParams {
    const void *W;
    void *Wp;            // nullable
    uint32_t *mask;      // nullable
    const float *scale;  // precomputed fl32(norm^alpha)
    struct LineResult *results;   // per-line thresholds (column lines only: a second, streaming kernel emits)
    int64_t rows, cols, ld;
    int64_t wpr;
    int64_t L;           // line length
    int64_t nlines;
    int64_t lpad;        // L rounded up to 8
    uint32_t k;          // survivors per line
    int scale_along_line;   // 1: scale[e] varies along the line; 0: scale[line]
};

// out[i] = fl32(norm[i]^alpha) for i < n, 0 for the padding up to npad (a multiple of 8, so that the selection
// kernel can read whole 8-element chunks)
__global__ void scale_vector_kernel(const float *__restrict__ norm, int64_t n, int64_t npad, int mode, float alpha,
                                    float *__restrict__ out)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = scale_from_norm(norm[i], mode, alpha);
    else if (i < npad) out[i] = 0.0f;
}

template <bool BF16>
__device__ __forceinline__ float abs_of(uint32_t raw)
{
    return BF16 ? __uint_as_float((raw & 0x7fffu) << 16) : __uint_as_float(raw & 0x7fffffffu);
}

// Adds 1 to bin `digit` of a shared-memory histogram for every lane with `active` set.  Lanes of the warp that hit
// the same bin are combined into one atomic (the top digits of a line are nearly all equal).
__device__ __forceinline__ void hist_add(uint32_t *h, uint32_t digit, bool active)
{
    const unsigned act = __ballot_sync(FULL_MASK, active);
    if (active) {
        const unsigned peers = __match_any_sync(act, digit);
        if ((threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(h + digit, (uint32_t)__popc(peers));
    }
}

struct LineState {
    unsigned long long tau64;   // threshold of the exact stage
    uint32_t tau32;             // threshold among the rounded products (bit pattern)
    uint32_t krem;              // survivors still to be taken at the current stage
    uint32_t neq;               // candidates in the last chosen bucket
    uint32_t exact;             // 1: rounded products tie across the cut, the exact stage decides
};

// One warp per line: finds the bucket (8-bit digit) that holds the krem-th largest candidate.
// Returns through lane-uniform values: the digit, the number of candidates in higher buckets, the bucket count.
__device__ __forceinline__ void find_bucket(const uint32_t *hist_line /* [nwarps][256] */, int nwarps, uint32_t krem, int lane,
                                            uint32_t &digit, uint32_t &greater, uint32_t &bucket)
{
    uint32_t cnt[8], lane_sum = 0u;
#pragma unroll
    for (int b = 0; b < 8; ++b) {
        uint32_t c = 0u;
        for (int w = 0; w < nwarps; ++w) c += hist_line[w * 256 + lane * 8 + b];
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
    const bool mine = above < krem && krem <= above + lane_sum;
    uint32_t d = 0u, g = 0u, bc = 0u;
    if (mine) {
#pragma unroll
        for (int b = 7; b >= 0; --b) {
            if (krem <= above + cnt[b]) { d = (uint32_t)(lane * 8 + b); g = above; bc = cnt[b]; break; }
            above += cnt[b];
        }
    }
    const uint32_t who = __ballot_sync(FULL_MASK, mine);
    const int src = who ? __ffs(who) - 1 : 0;
    digit = __shfl_sync(FULL_MASK, d, src);
    greater = __shfl_sync(FULL_MASK, g, src);
    bucket = __shfl_sync(FULL_MASK, bc, src);
}

// LINE_IS_ROW: the CTA's line is matrix row b.  Otherwise its two lines are the matrix columns 2b, 2b+1 (one 4- or
// 8-byte load per row fetches both).  Every thread works on all lines of its CTA.
//
// Stage A selects on p = fl32(|w| * scale) (rounding is monotone, so p decides every pair whose rounded products
// differ): four 8-bit passes give the threshold tau32.  If exactly the needed number of products equal tau32, all of
// them stay and the line is done.  Otherwise stage B repeats the selection among those equal products with the exact
// double products as keys (eight passes), and the emit pass breaks remaining exact ties towards the lower index.
template <bool BF16, bool LINE_IS_ROW>
__global__ void __launch_bounds__(LINE_IS_ROW ? 256 : 512) select_unstructured_kernel(const SelectParams p)
{
    constexpr int U_THREADS = LINE_IS_ROW ? 256 : 512;   // row lines: 3 CTAs per SM; column lines: one CTA (2 lines) per SM
    constexpr int U_WARPS = U_THREADS / 32;
    using elem_t = typename std::conditional<BF16, uint16_t, uint32_t>::type;
    constexpr int U_LINES = LINE_IS_ROW ? 1 : 2;
    extern __shared__ __align__(16) unsigned char u_smem[];
    elem_t *line_mem = reinterpret_cast<elem_t *>(u_smem);                       // [U_LINES][lpad]
    uint32_t *hist = reinterpret_cast<uint32_t *>(u_smem + (size_t)U_LINES * p.lpad * sizeof(elem_t));   // [U_LINES][U_WARPS][256]
    __shared__ LineState st[U_LINES];
    __shared__ uint32_t s_warp_tot[U_WARPS];
    __shared__ uint32_t s_any_exact;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t line0 = (int64_t)blockIdx.x * U_LINES;
    const int nl = (int)((p.nlines - line0) < U_LINES ? (p.nlines - line0) : U_LINES);
    const int64_t nchunks = p.lpad >> 3;
    constexpr int TPL = U_THREADS;                                              // threads per line
    constexpr int my_first = 0;
    constexpr int my_count = U_LINES;
    const int tau = tid;
    const int64_t nbatches = (nchunks + TPL - 1) / TPL;

    // ---------------------------------------------------------------- phase 0: lines -> shared memory
    if constexpr (LINE_IS_ROW) {
        // 16-byte loads: rows are 16-byte aligned and padded to whole vectors by the ld rule; elements past L
        // that a vector drags in are never used (every consumer checks the index against L)
        const uint4 *src = reinterpret_cast<const uint4 *>(static_cast<const elem_t *>(p.W) + line0 * p.ld);
        uint4 *dst = reinterpret_cast<uint4 *>(line_mem);
        constexpr int EPV = 16 / sizeof(elem_t);
        const int64_t nvec = (p.L + EPV - 1) / EPV;
        for (int64_t v = tid; v < (int64_t)(p.lpad / EPV); v += U_THREADS) dst[v] = v < nvec ? __ldcs(src + v) : make_uint4(0u, 0u, 0u, 0u);
    } else {
        const elem_t *src = static_cast<const elem_t *>(p.W) + line0;            // column line0 of row r at src[r * ld]
        for (int64_t r = tid; r < p.lpad; r += U_THREADS) {
#pragma unroll
            for (int ln = 0; ln < U_LINES; ++ln)
                line_mem[ln * p.lpad + r] = (r < p.L && ln < nl) ? src[r * p.ld + ln] : (elem_t)0;
        }
    }
    if (tid < U_LINES) { st[tid].tau64 = 0ull; st[tid].tau32 = 0u; st[tid].krem = p.k; st[tid].neq = 0u; st[tid].exact = 0u; }
    if (tid == 0) s_any_exact = 0u;
    __syncthreads();

    // the 8 rounded products of chunk q of line ln (0 for positions past the line's end)
    auto products = [&](int ln, int64_t q, float line_scale, float (&pf)[8]) {
        float sc[8];
        if (p.scale_along_line) {
            const float4 s0 = __ldg(reinterpret_cast<const float4 *>(p.scale + q * 8));
            const float4 s1 = __ldg(reinterpret_cast<const float4 *>(p.scale + q * 8) + 1);   // the vector is padded to 8
            sc[0] = s0.x; sc[1] = s0.y; sc[2] = s0.z; sc[3] = s0.w; sc[4] = s1.x; sc[5] = s1.y; sc[6] = s1.z; sc[7] = s1.w;
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) sc[j] = line_scale;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) pf[j] = __fmul_rn(abs_of<BF16>(line_mem[ln * p.lpad + q * 8 + j]), sc[j]);
    };

    // ---------------------------------------------------------------- stage A: radix select on the rounded products
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = tid; i < U_LINES * U_WARPS * 256; i += U_THREADS) hist[i] = 0u;
        __syncthreads();
        const uint32_t known = shift == 24 ? 0u : (~0u << (shift + 8));
        for (int m = 0; m < my_count; ++m) {
            const int ln = my_first + m;
            const bool live = ln < nl;
            const uint32_t prefix = live ? st[ln].tau32 : 0u;
            const float line_scale = (!live || p.scale_along_line) ? 0.0f : p.scale[line0 + ln];
            uint32_t *h = hist + ((live ? ln : 0) * U_WARPS + warp) * 256;
            for (int64_t bt = 0; bt < nbatches; ++bt) {          // same trip count for every lane (warp-wide votes inside)
                const int64_t q = bt * TPL + tau;
                const bool have = live && q < nchunks;
                float pf[8];
                if (have) products(ln, q, line_scale, pf);
                if (shift == 24) {
                    // first pass: every element is a candidate and the top byte (sign and high exponent bits) is the
                    // same for most of a line, so whole chunks are counted at once and merged across the warp
                    uint32_t d0 = 0u;
                    bool same = have && (q * 8 + 7 < p.L);
                    if (have) {
                        d0 = __float_as_uint(pf[0]) >> 24;
#pragma unroll
                        for (int j = 1; j < 8; ++j) same = same && ((__float_as_uint(pf[j]) >> 24) == d0);
                    }
                    if (__all_sync(FULL_MASK, same || !have)) {
                        const unsigned act = __ballot_sync(FULL_MASK, have);
                        if (have) {
                            const unsigned peers = __match_any_sync(act, d0);
                            if (lane == __ffs(peers) - 1) atomicAdd(h + d0, 8u * (uint32_t)__popc(peers));
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            hist_add(h, have ? (__float_as_uint(pf[j]) >> 24) : 0u, have && (q * 8 + j < p.L));
                    }
                } else if (have) {
                    // later passes: few candidates, spread over many bins: plain atomics
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t key = __float_as_uint(pf[j]);
                        if ((q * 8 + j < p.L) && (((key ^ prefix) & known) == 0u)) atomicAdd(h + ((key >> shift) & 0xffu), 1u);
                    }
                }
            }
        }
        __syncthreads();
        if (warp < nl) {
            uint32_t digit, greater, bucket;
            find_bucket(hist + warp * U_WARPS * 256, U_WARPS, st[warp].krem, lane, digit, greater, bucket);
            if (lane == 0) {
                st[warp].tau32 |= digit << shift;
                st[warp].krem -= greater;
                if (shift == 0) {
                    st[warp].neq = bucket;
                    if (bucket != st[warp].krem) { st[warp].exact = 1u; s_any_exact = 1u; }
                }
            }
        }
        __syncthreads();
    }

    // ---------------------------------------------------------------- stage B: exact keys among the tied products
    if (s_any_exact) {
        for (int shift = 56; shift >= 0; shift -= 8) {
            for (int i = tid; i < U_LINES * U_WARPS * 256; i += U_THREADS) hist[i] = 0u;
            __syncthreads();
            const unsigned long long known = shift == 56 ? 0ull : (~0ull << (shift + 8));
            for (int m = 0; m < my_count; ++m) {
                const int ln = my_first + m;
                const bool live = ln < nl && st[ln < nl ? ln : 0].exact;
                const uint32_t t32 = live ? st[ln].tau32 : 0u;
                const unsigned long long prefix = live ? st[ln].tau64 : 0ull;
                const float line_scale = (!live || p.scale_along_line) ? 0.0f : p.scale[line0 + ln];
                uint32_t *h = hist + ((live ? ln : 0) * U_WARPS + warp) * 256;
                for (int64_t bt = 0; bt < nbatches; ++bt) {
                    const int64_t q = bt * TPL + tau;
                    const bool have = live && q < nchunks;
                    float pf[8];
                    if (have) products(ln, q, line_scale, pf);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        bool cand = have && (q * 8 + j < p.L) && __float_as_uint(pf[j]) == t32;
                        unsigned long long key = 0ull;
                        if (cand) {
                            const float sc = p.scale_along_line ? __ldg(p.scale + q * 8 + j) : line_scale;
                            key = (unsigned long long)__double_as_longlong((double)abs_of<BF16>(line_mem[ln * p.lpad + q * 8 + j]) * (double)sc);
                            cand = ((key ^ prefix) & known) == 0ull;
                        }
                        if (cand) atomicAdd(h + (uint32_t)((key >> shift) & 0xffull), 1u);
                    }
                }
            }
            __syncthreads();
            if (warp < nl && st[warp].exact) {
                uint32_t digit, greater, bucket;
                find_bucket(hist + warp * U_WARPS * 256, U_WARPS, st[warp].krem, lane, digit, greater, bucket);
                if (lane == 0) {
                    st[warp].tau64 |= (unsigned long long)digit << shift;
                    st[warp].krem -= greater;
                }
            }
            __syncthreads();
        }
    }

    if constexpr (!LINE_IS_ROW) {
        // column lines: publish the thresholds; select_emit_cols_kernel writes the outputs with coalesced rows.
        // The loop below then only locates the cut among exact ties (skipped when no line of the CTA has any).
        if (tid < nl) {
            LineResult r;
            r.tau64 = st[tid].tau64; r.cut = -1; r.tau32 = st[tid].tau32; r.exact = st[tid].exact;
            p.results[line0 + tid] = r;
        }
        __syncthreads();
        if (!s_any_exact) return;
    }
    // ---------------------------------------------------------------- emit in index order
    for (int m = 0; m < my_count; ++m) {
        const int ln = my_first + m;
        const bool live = ln < nl;
        const LineState ls = st[live ? ln : 0];
        const float line_scale = (!live || p.scale_along_line) ? 0.0f : p.scale[line0 + ln];
        uint32_t base = 0u;                                  // exact ties seen before this batch
        for (int64_t bt = 0; bt < nbatches; ++bt) {
            const int64_t q = bt * TPL + tau;
            const bool have = live && q < nchunks;
            uint32_t keep = 0u, eq = 0u;
            if (have) {
                float pf[8];
                products(ln, q, line_scale, pf);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (q * 8 + j < p.L) {
                        const uint32_t key = __float_as_uint(pf[j]);
                        if (key > ls.tau32) {
                            keep |= 1u << j;
                        } else if (key == ls.tau32) {
                            if (!ls.exact) {
                                keep |= 1u << j;             // all products equal to the threshold stay
                            } else {
                                const float sc = p.scale_along_line ? __ldg(p.scale + q * 8 + j) : line_scale;
                                const unsigned long long k64 = (unsigned long long)__double_as_longlong(
                                    (double)abs_of<BF16>(line_mem[ln * p.lpad + q * 8 + j]) * (double)sc);
                                if (k64 > ls.tau64) keep |= 1u << j;
                                else if (k64 == ls.tau64) eq |= 1u << j;
                            }
                        }
                    }
                }
            }
            if (s_any_exact) {
                // exclusive prefix of the exact-tie counts over the line's threads, in thread (= index) order
                const uint32_t mycnt = __popc(eq);
                uint32_t incl = mycnt;
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                    const uint32_t t = __shfl_up_sync(FULL_MASK, incl, off);
                    if (lane >= off) incl += t;
                }
                if (lane == 31) s_warp_tot[warp] = incl;
                __syncthreads();
                const int w_first = 0;
                uint32_t before = base, batch_total = 0u;
                for (int w = 0; w < TPL / 32; ++w) {
                    const uint32_t t = s_warp_tot[w_first + w];
                    if (w_first + w < warp) before += t;
                    batch_total += t;
                }
                __syncthreads();
                uint32_t rank = before + incl - mycnt;       // exact ties with a lower index than this thread's first
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if ((eq >> j) & 1u) {
                        if (rank < ls.krem) keep |= 1u << j;
                        if constexpr (!LINE_IS_ROW) {
                            if (ls.exact && rank + 1 == ls.krem) p.results[line0 + ln].cut = q * 8 + j;   // last exact tie that stays
                        }
                        ++rank;
                    }
                }
                base += batch_total;
            }

            if (have) {
                const int64_t e0 = q * 8;
                const int64_t left = p.L - e0;
                const int nvalid = left >= 8 ? 8 : (int)left;
                if constexpr (LINE_IS_ROW) {
                    const int64_t r = line0 + ln;
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
                }
            }
        }
    }
}

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

template <bool BF16>
__global__ void __launch_bounds__(256) select_emit_cols_kernel(const EmitParams p)
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
                tau[j] = p.results[c0 + j].tau32;
                exact_cols |= (p.results[c0 + j].exact ? 1u : 0u) << j;
                if (!p.scale_per_row) sc[j] = p.scale[c0 + j];
            }
        }
        for (int i = 0; i < 32; ++i) {
            const int64_t r = rb * 32 + i;
            if (r >= p.rows) break;                     // warp-uniform
            Chunk<BF16> ch;
            if (nvalid > 0) chunk_load<BF16>(ch, p.W, r * p.ld + c0, nvalid);
            else chunk_zero<BF16>(ch);
            const float rs = p.scale_per_row ? __ldg(p.scale + r) : 0.0f;
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
                        const LineResult res = p.results[c0 + j];
                        const unsigned long long k64 = (unsigned long long)__double_as_longlong((double)a * (double)s);
                        k = k64 > res.tau64 || (k64 == res.tau64 && (long long)r <= res.cut);
                    }
                }
                keep |= (k && j < nvalid ? 1u : 0u) << j;
            }
            const uint32_t word = quad_pack_bytes(keep, lane);
            if (nvalid > 0) {
                if (p.mask && (lane & 3) == 0) p.mask[r * p.wpr + (c0 >> 5)] = word;
                if (p.Wp) {
                    chunk_apply_mask<BF16>(ch, keep);
                    chunk_store<BF16>(ch, p.Wp, r * p.ld + c0, nvalid);
                }
            }
        }
    }
}

int device_sm_count();   // dass_abi.cu

size_t select_smem_bytes(int64_t L, bool bf16, bool line_is_row)
{
    const int64_t lpad = (L + 7) / 8 * 8;
    const size_t lines = line_is_row ? 1 : 2;
    const size_t warps = line_is_row ? 8 : 16;
    return lines * lpad * (bf16 ? 2 : 4) + lines * warps * 256 * sizeof(uint32_t);
}

template <bool BF16, bool ROW>
static cudaError_t launch_select(const SelectParams &p, size_t smem, cudaStream_t st)
{
    cudaError_t e = cudaFuncSetAttribute(select_unstructured_kernel<BF16, ROW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    constexpr int lines = ROW ? 1 : 2;
    const int64_t grid = (p.nlines + lines - 1) / lines;
    select_unstructured_kernel<BF16, ROW><<<(unsigned)grid, ROW ? 256 : 512, smem, st>>>(p);
    return cudaGetLastError();
}

size_t select_results_bytes(int64_t cols) { return ((size_t)cols * sizeof(LineResult) + 31) / 32 * 32; }

cudaError_t select_unstructured_launch(const void *W, int64_t rows, int64_t cols, int64_t ld, bool bf16,
                                       const float *norm, bool norm_cols, float alpha, uint32_t k, bool line_is_row,
                                       uint32_t *mask_bits, void *W_pruned, void *workspace, cudaStream_t st)
{
    // workspace: [per-column results][scale vector padded to 8]
    LineResult *results = static_cast<LineResult *>(workspace);
    float *scale_ws = reinterpret_cast<float *>(static_cast<unsigned char *>(workspace) + select_results_bytes(cols));
    const int64_t n_norm = norm_cols ? cols : rows;
    const int64_t n_pad = (n_norm + 7) / 8 * 8;
    scale_vector_kernel<<<(unsigned)((n_pad + 255) / 256), 256, 0, st>>>(norm, n_norm, n_pad, (int)scale_mode_for(alpha), alpha, scale_ws);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    SelectParams p;
    p.W = W; p.Wp = W_pruned; p.mask = mask_bits; p.scale = scale_ws; p.results = results;
    p.rows = rows; p.cols = cols; p.ld = ld;
    p.wpr = (cols + 31) / 32;
    p.L = line_is_row ? cols : rows;
    p.nlines = line_is_row ? rows : cols;
    p.lpad = (p.L + 7) / 8 * 8;
    p.k = k;
    p.scale_along_line = (line_is_row == norm_cols) ? 1 : 0;   // the norm index runs along the line
    const size_t smem = select_smem_bytes(p.L, bf16, line_is_row);
    if (line_is_row) {
        if (mask_bits) {   // the kernel writes whole bytes of real columns; the padding of each mask row must read 0
            e = cudaMemsetAsync(mask_bits, 0, (size_t)rows * p.wpr * sizeof(uint32_t), st);
            if (e != cudaSuccess) return e;
        }
        return bf16 ? launch_select<true, true>(p, smem, st) : launch_select<false, true>(p, smem, st);
    }
    e = bf16 ? launch_select<true, false>(p, smem, st) : launch_select<false, false>(p, smem, st);
    if (e != cudaSuccess) return e;
    EmitParams q;
    q.W = W; q.Wp = W_pruned; q.mask = mask_bits; q.scale = scale_ws; q.results = results;
    q.rows = rows; q.cols = cols; q.ld = ld; q.wpr = p.wpr;
    q.col_blocks = (cols + 255) / 256;
    q.row_blocks = (rows + 31) / 32;
    q.scale_per_row = norm_cols ? 0 : 1;
    const int64_t want = (q.col_blocks * q.row_blocks + 7) / 8;
    const int64_t cap = (int64_t)device_sm_count() * 8;
    const int grid = (int)(want < cap ? want : cap);
    if (bf16) select_emit_cols_kernel<true><<<grid, 256, 0, st>>>(q);
    else select_emit_cols_kernel<false><<<grid, 256, 0, st>>>(q);
    return cudaGetLastError();
}

}  // namespace dass

using namespace dass;

extern "C" dass_status dass_select_workspace_bytes(int64_t rows, int64_t cols, dass_axis norm_axis, size_t *bytes)
{
    if (!bytes) return DASS_ERR_NULL;
    if (norm_axis != DASS_AXIS_ROWS && norm_axis != DASS_AXIS_COLS) return DASS_ERR_DTYPE;
    if (rows < 1 || cols < 1) return DASS_ERR_SHAPE;
    const int64_t n = norm_axis == DASS_AXIS_ROWS ? rows : cols;
    *bytes = select_results_bytes(cols) + (size_t)((n + 7) / 8 * 8) * sizeof(float);
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
    if (select_smem_bytes(L, bf16, false) > (size_t)220 * 1024) return DASS_ERR_UNSUPPORTED;   // two lines must fit in shared memory
    const int64_t n_prune = (int64_t)std::floor(sparsity * (double)L);
    const uint32_t k = (uint32_t)(L - n_prune);
    if (select_unstructured_launch(W, rows, cols, ld, bf16, norm, norm_axis == DASS_AXIS_COLS, alpha, k, line_is_row,
                                   mask_bits, W_pruned, workspace,
                                   static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return DASS_ERR_CUDA;
    return DASS_OK;
}
