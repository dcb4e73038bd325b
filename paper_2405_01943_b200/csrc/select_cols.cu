// Unstructured selection, lines that are matrix columns (input-balanced: a column of Wg / Wu): the kernel that
// decides every column of a strip, up to one histogram bin (bf16) or completely.
#include "select_common.cuh"

namespace dass {

// ---------------------------------------------------------------- lines that are matrix columns
// One CTA per strip of 8 adjacent columns (16 bytes of every row for bf16, 32 for f32).  The strip is not cached: the
// sweep of the sampled bracket reads it once (bf16: through bulk tensor copies), and every pass of the radix select,
// where a column needs it, reads it again with one vector load per row and thread (mostly from L2).  The kernel
// publishes a LineResult per column: the bin that holds the cut (bf16), or the exact rule (tau32, exact, tau64, cut).
constexpr int COL_THREADS = 512;                // two CTAs per SM: one sweeps while the other samples, picks its bins or waits
constexpr int COL_SAMPLE = SELECT_SAMPLE;       // evenly spaced rows of a strip that place its columns' brackets
constexpr int COL_LINES = 8;
constexpr int COL_COPIES = 1;                   // histogram copies per column (3 measured slower, as for rows)

// ALONG: the scale varies along the columns (one per row) rather than being one number per column.
// TMA (bf16, at least 8 columns): the sweep of the sampled bracket receives the strip through bulk tensor copies --
// SR_STAGE_ROWS rows of 16 bytes per stage, one stage in flight while the other is worked on -- instead of one 16-byte load per thread from 1024
// different cache lines per warp instruction pair, which kept the load/store pipe busier than the arithmetic.
constexpr int HSTRIDE = BBINS + 32;                      // a column's bins of the bracket sweep, then one idle word per lane
constexpr int SR_STAGES = 2;
constexpr int SR_BOX_ROWS = 256;                         // rows of one bulk copy (a box dimension is at most 256)
constexpr int SR_STAGE_ROWS = 2048;                      // rows of one stage: SR_RPT per thread
constexpr int SR_RPT = SR_STAGE_ROWS / COL_THREADS;
constexpr uint32_t SR_STAGE_BYTES = SR_STAGE_ROWS * 16u;

template <bool BF16, bool ALONG, bool TMA>
__global__ void __launch_bounds__(COL_THREADS, 2) select_cols_kernel(const __grid_constant__ CUtensorMap map_w, const SelectParams p)
{
    static_assert(!TMA || BF16, "the bulk-copy sweep is written for bf16 strips");
    using elem_t = typename std::conditional<BF16, uint16_t, uint32_t>::type;
    extern __shared__ __align__(16) unsigned char u_smem[];
    uint32_t *hist = reinterpret_cast<uint32_t *>(u_smem);       // [COL_LINES][COL_COPIES][HBINS]
    __shared__ Line st[COL_LINES];
    __shared__ uint32_t s_long;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t c0 = (int64_t)blockIdx.x * COL_LINES;
    const int nl = (int)((p.cols - c0) < COL_LINES ? (p.cols - c0) : COL_LINES);
    const uint32_t idx_top = (uint32_t)((1ull << p.idx_bits) - 1ull);
    const elem_t *strip = static_cast<const elem_t *>(p.W) + c0;

    if (tid < COL_LINES) line_init(st[tid], p.k);
    if (tid == 0) s_long = 0u;
    float col_scale[COL_LINES];
#pragma unroll
    for (int j = 0; j < COL_LINES; ++j) col_scale[j] = (!p.scale_along_line && j < nl) ? DASS_LD(&p.scale[c0 + j]) : 0.0f;

    // One pass over the strip: UNROLL rows per thread are loaded before any is counted, so that several
    // L2 round trips are in flight per thread.
    constexpr int UNROLL = BF16 ? 4 : 2;
    uint32_t *my_hist = hist + (lane % COL_COPIES) * HBINS;
    auto count_pass = [&](auto mode_tag, const Sched &sc, const uint32_t (&t32)[COL_LINES]) {
        constexpr int MODE = decltype(mode_tag)::value;
        for (int64_t r0 = tid; r0 < p.L; r0 += (int64_t)UNROLL * COL_THREADS) {
            Chunk<BF16> ch[UNROLL];
            float row_scale[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int64_t r = r0 + (int64_t)u * COL_THREADS;
                chunk_zero<BF16>(ch[u]);
                row_scale[u] = 0.0f;
                if (r < p.L) {
                    // the row pitch is a multiple of 16 bytes and c0 of 8 elements: aligned vectors inside the row's
                    // pitch (an f32 row is padded to 4 elements only: its second vector is read when it holds a column)
                    const uint4 *src = reinterpret_cast<const uint4 *>(strip + r * p.ld);
                    const uint4 v0 = DASS_LD_G(src);
                    ch[u].w[0] = v0.x; ch[u].w[1] = v0.y; ch[u].w[2] = v0.z; ch[u].w[3] = v0.w;
                    if constexpr (!BF16) {
                        if (nl > 4) {
                            const uint4 v1 = DASS_LD_G(src + 1);
                            ch[u].w[4] = v1.x; ch[u].w[5] = v1.y; ch[u].w[6] = v1.z; ch[u].w[7] = v1.w;
                        }
                    }
                    if (p.scale_along_line) row_scale[u] = DASS_LD_G(p.scale + r);
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int64_t r = r0 + (int64_t)u * COL_THREADS;
                if (r < p.L) {
#pragma unroll
                    for (int j = 0; j < COL_LINES; ++j) {
                        const float s = p.scale_along_line ? row_scale[u] : col_scale[j];
                        if (MODE != COUNT_ALL || j < nl)
                            count_element<MODE>(my_hist + j * (COL_COPIES * HBINS), st[j], t32[j], chunk_float<BF16>(ch[u], j), s, (uint32_t)r, sc, idx_top);
                    }
                }
            }
        }
    };

    // ---------------------------------------------------------------- sampled bracket (see the top of the file)
    constexpr bool DEFER = BF16;                     // bf16: the column is published at its bin and the emit pass sets the bin's elements aside
    __shared__ FastLine fl[COL_LINES];
    __shared__ CandSet cand[DEFER ? 1 : COL_LINES];
    __shared__ uint32_t s_over[COL_LINES];           // sample keys above a column's window
    bool any_pending = true;
    if (tid < COL_LINES) { fl[tid].ok = 0u; fl[tid].lo = 0u; fl[tid].hi = 0u; }     // past the matrix edge: an empty bracket
    if (p.L >= FAST_MIN_L && p.L <= FAST_MAX_L) {    // the same for every thread
        const uint32_t hist_s = smem_u32(hist);
        // the ring of the bulk-copy sweep, behind the histograms (128-byte aligned), and its barriers
        uint8_t *ring_mem = u_smem + (size_t)COL_LINES * HSTRIDE * sizeof(uint32_t);
        ring_mem += (128u - (smem_u32(ring_mem) & 127u)) & 127u;
        const uint32_t ring_s = smem_u32(ring_mem), bars_s = ring_s + SR_STAGES * SR_STAGE_BYTES;
        const int n_it = (int)((p.L + SR_STAGE_ROWS - 1) / SR_STAGE_ROWS);
        auto ring_issue = [&](int it) {              // one thread: the rows from it * SR_STAGE_ROWS into stage it % SR_STAGES
            const uint32_t bar = bars_s + 8u * (uint32_t)(it % SR_STAGES);
            const uint32_t dst = ring_s + (uint32_t)(it % SR_STAGES) * SR_STAGE_BYTES;
            mbar_arrive_expect_tx(bar, SR_STAGE_BYTES);
#pragma unroll
            for (int b = 0; b < SR_STAGE_ROWS / SR_BOX_ROWS; ++b)
                tma_load_2d(dst + (uint32_t)(b * SR_BOX_ROWS * 16), &map_w, bar, (int)c0, it * SR_STAGE_ROWS + b * SR_BOX_ROWS);
        };
        if constexpr (TMA) {                         // the first stages travel while the sample is taken
            if (tid == 0) {
#pragma unroll
                for (int s_ = 0; s_ < SR_STAGES; ++s_) mbar_init(bars_s + 8u * s_, 1);
                asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
                for (int it = 0; it < SR_STAGES - 1 && it < n_it; ++it) ring_issue(it);
            }
        }
        // loads one row of the strip (the vector loads of count_pass)
        auto load_row = [&](int64_t r, Chunk<BF16> &ch) {
            const uint4 *src = reinterpret_cast<const uint4 *>(strip + r * p.ld);
            const uint4 v0 = DASS_LD_G(src);
            ch.w[0] = v0.x; ch.w[1] = v0.y; ch.w[2] = v0.z; ch.w[3] = v0.w;
            if constexpr (!BF16) {
                ch.w[4] = ch.w[5] = ch.w[6] = ch.w[7] = 0u;
                if (nl > 4) {
                    const uint4 v1 = DASS_LD_G(src + 1);
                    ch.w[4] = v1.x; ch.w[5] = v1.y; ch.w[6] = v1.z; ch.w[7] = v1.w;
                }
            }
        };
        // visits every row of the strip, UNROLL rows of a thread in flight: f(column, signed weight, scale, row)
        auto sweep = [&](auto &&f) {
            for (int64_t r0 = tid; r0 < p.L; r0 += (int64_t)UNROLL * COL_THREADS) {
                Chunk<BF16> ch[UNROLL];
                float row_scale[UNROLL];
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const int64_t r = r0 + (int64_t)u * COL_THREADS;
                    chunk_zero<BF16>(ch[u]);
                    row_scale[u] = 0.0f;
                    if (r < p.L) {
                        load_row(r, ch[u]);
                        if constexpr (ALONG) row_scale[u] = DASS_LD_G(p.scale + r);
                    }
                }
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const int64_t r = r0 + (int64_t)u * COL_THREADS;
                    if (r < p.L) {
#pragma unroll
                        for (int j = 0; j < COL_LINES; ++j)
                            f(j, chunk_float<BF16>(ch[u], j), ALONG ? row_scale[u] : col_scale[j], r);
                    }
                }
            }
        };
        uint32_t *ehist = hist;                      // [COL_LINES][256] exponent counts of the sample, before the bins
        uint32_t *fhist = hist + COL_LINES * 256;    // [COL_LINES][FINE_BINS] the sample inside each column's window
        for (int i = tid; i < COL_LINES * (256 + FINE_BINS); i += COL_THREADS) hist[i] = 0u;
        if (tid < COL_LINES) s_over[tid] = 0u;
        __syncthreads();
        constexpr int SPT = COL_SAMPLE / COL_THREADS;
        uint32_t skey[SPT][COL_LINES];               // the sample: SPT rows per thread, all of the strip's columns
#pragma unroll
        for (int u = 0; u < SPT; ++u) {
            const int64_t r = ((int64_t)(tid + u * COL_THREADS) * p.L) / COL_SAMPLE;
            Chunk<BF16> ch;
            load_row(r, ch);
            float rs = 0.0f;
            if constexpr (ALONG) rs = DASS_LD_G(p.scale + r);
#pragma unroll
            for (int j = 0; j < COL_LINES; ++j) skey[u][j] = product_key(chunk_float<BF16>(ch, j), ALONG ? rs : col_scale[j]);
        }
#pragma unroll
        for (int u = 0; u < SPT; ++u) {
#pragma unroll
            for (int j = 0; j < COL_LINES; ++j) {
                // a warp's keys share a few exponents: one update per distinct exponent
                const uint32_t e = skey[u][j] >> 23;
                const uint32_t same = __match_any_sync(FULL_MASK, e);
                if (lane == __ffs(same) - 1) atomicAdd(ehist + j * 256 + e, (uint32_t)__popc(same));
            }
        }
        __syncthreads();
        const int target = (int)win_target(p.k, p.L, COL_SAMPLE);
        if (warp < nl) window_from_exponents(ehist + warp * 256, fl[warp], (uint32_t)target, lane);
        __syncthreads();
#pragma unroll
        for (int u = 0; u < SPT; ++u) {
#pragma unroll
            for (int j = 0; j < COL_LINES; ++j) {
                if (j < nl) {
                    const uint32_t wlo = fl[j].lo, off = skey[u][j] - wlo;
                    if (off < WIN_SPAN) atomicAdd(fhist + j * FINE_BINS + (off >> FINE_SHIFT), 1u);
                    else if (skey[u][j] > wlo) atomicAdd(&s_over[j], 1u);
                }
            }
        }
        __syncthreads();
        if (warp < nl) bracket_from_fine(fhist + warp * FINE_BINS, s_over[warp], fl[warp], target, p.margin, lane);
        __syncthreads();
        bool lost = false;                           // a bounded wait of the bulk-copy sweep ran out
        uint32_t mul = 0xffffffffu;                  // one bin width for the strip: the widest bracket's
#pragma unroll
        for (int j = 0; j < COL_LINES; ++j) mul = (j < nl && fl[j].mul < mul) ? fl[j].mul : mul;
        for (int i = tid; i < COL_LINES * HSTRIDE; i += COL_THREADS) hist[i] = 0u;
        __syncthreads();
        if (tid < nl) { fl[tid].mul = mul; fl[tid].hi = fl[tid].lo + bin_start((uint32_t)BBINS, mul); }
        {   // first pass: the elements inside a column's bracket go to its histogram (predicated: the other lanes cost
            // the shared-memory pipe nothing), those below it are counted, those above it follow from the length
            uint32_t lo[COL_LINES], below[COL_LINES];
#pragma unroll
            for (int j = 0; j < COL_LINES; ++j) {
                lo[j] = fl[j].lo;                    // (a column past the matrix edge fills bins nobody reads)
                below[j] = 0u;
            }
            // every lane updates a counter: its element's bin inside the bracket (the bracket spans all BBINS bins), else a
            // word of its own behind the column's bins that nobody reads
            const uint32_t idle_bin = (uint32_t)(BBINS + lane);
            auto count_key = [&](auto jc, uint32_t key) {                 // jc: the column, a compile-time constant
                constexpr int J = decltype(jc)::value;
                const uint32_t off = key - lo[J];                         // keys are below 2^31: the top bit says "below lo"
                asm volatile("red.shared.add.u32 [%0+%1], 1;" ::"r"(hist_s + (min(__umulhi(off, mul), idle_bin) << 2)), "n"(J * HSTRIDE * 4) : "memory");
                below[J] = __umulhi(off, 2u) + below[J];
            };
            auto visit = [&](int j, float wf, float sc_, int64_t) {
                const uint32_t off = product_key(wf, sc_) - lo[j];
                asm volatile("red.shared.add.u32 [%0], 1;" ::"r"(hist_s + (uint32_t)(j * HSTRIDE * 4) + (min(__umulhi(off, mul), idle_bin) << 2)) : "memory");
                below[j] = __umulhi(off, 2u) + below[j];
            };
            if constexpr (TMA) {
                for (int it = 0; it < n_it; ++it) {
                    // the stage read one iteration ago is free (every thread passed that iteration's barrier)
                    if (tid == 0 && it + SR_STAGES - 1 < n_it) ring_issue(it + SR_STAGES - 1);
                    const int64_t r0 = (int64_t)it * SR_STAGE_ROWS + tid;
                    float rs[SR_RPT];
#pragma unroll
                    for (int u = 0; u < SR_RPT; ++u) {
                        rs[u] = 0.0f;
                        if constexpr (ALONG) rs[u] = r0 + u * COL_THREADS < p.L ? DASS_LD_G(p.scale + r0 + u * COL_THREADS) : 0.0f;
                    }
                    const bool ok = slot_wait(bars_s + 8u * (uint32_t)(it % SR_STAGES), (uint32_t)((it / SR_STAGES) & 1));
                    uint4 v[SR_RPT];
#pragma unroll
                    for (int u = 0; u < SR_RPT; ++u)
                        v[u] = *reinterpret_cast<const uint4 *>(ring_mem + (size_t)(it % SR_STAGES) * SR_STAGE_BYTES + (size_t)(u * COL_THREADS + tid) * 16);
                    if (__syncthreads_or(ok ? 0 : 1)) { lost = true; break; }
#pragma unroll
                    for (int u = 0; u < SR_RPT; ++u) {
                        if (r0 + u * COL_THREADS < p.L) {    // rows past the end arrive as zeros and are not counted
                            const uint32_t w4[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                            static_for<COL_LINES>([&](auto jc) {
                                constexpr int J = decltype(jc)::value;
                                const float sv = ALONG ? rs[u] : col_scale[J];
                                count_key(jc, __float_as_uint((J & 1) ? prod_hi(w4[J >> 1], sv) : prod_lo(w4[J >> 1], sv)));
                            });
                        }
                    }
                }
                if (lost) {                          // recorded; the copies in flight get one more bounded chance to land,
                    if (tid == 0) {                  // and the radix select (plain loads) decides the strip
                        if (p.status) atomicMax(p.status, (int)DASS_ERR_TIMEOUT);
                        for (int s_ = 0; s_ < SR_STAGES; ++s_) { slot_wait(bars_s + 8u * s_, 0u); slot_wait(bars_s + 8u * s_, 1u); }
                    }
                }
            } else {
                sweep(visit);
            }
#pragma unroll
            for (int j = 0; j < COL_LINES; ++j) {
                uint32_t a = below[j];
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(FULL_MASK, a, off);
                if (lane == 0 && a && j < nl) atomicAdd(&fl[j].below, a);
            }
        }
        __syncthreads();
        if (warp < nl) bracket_pick_bin(hist + warp * HSTRIDE, fl[warp], p.k, lane, p.L);
        __syncthreads();
        if (lost) {   // the same for every thread: the counts are incomplete, and copies may still land in the ring,
                      // which the radix select would use as its histograms: the strip is given up (every element stays)
            if (tid < nl) {
                LineResult r;
                r.tau32 = 0u; r.exact = 0u; r.tau64 = 0ull; r.cut = 0ll;
                DASS_ST(&p.results[c0 + tid], r);
                if (p.cand_count) DASS_ST(&p.cand_count[c0 + tid], 0u);
            }
            return;
        }
        if constexpr (DEFER) {
            if (tid < nl && fl[tid].ok) {            // published at the bin; nothing set aside yet
                LineResult r;
                r.tau32 = fl[tid].bhi; r.exact = LINE_BIN;
                r.tau64 = (unsigned long long)fl[tid].blo | ((unsigned long long)fl[tid].krem2 << 32);
                r.cut = (long long)fl[tid].bucket;
                fl[tid].res = r;
            }
        } else {   // second pass: the elements of each column's bin are collected and ranked here
            uint32_t blo[COL_LINES], bw[COL_LINES];
            uint32_t some = 0u;
#pragma unroll
            for (int j = 0; j < COL_LINES; ++j) {
                const bool live = j < nl && fl[j].ok;
                blo[j] = live ? fl[j].blo : 0u;
                bw[j] = live ? fl[j].bhi - fl[j].blo : 0u;
                some |= live ? 1u : 0u;
            }
            if (some) {                              // the same for every thread
                sweep([&](int j, float wf, float sc_, int64_t r) {
                    const uint32_t key = product_key(wf, sc_);
                    if (key - blo[j] < bw[j]) {
                        const uint32_t slot = atomicAdd(&fl[j].ncoll, 1u);
                        if (slot < (uint32_t)CAND_CAP) {
                            cand[j].key[slot] = key; cand[j].idx[slot] = (uint32_t)r; cand[j].k64[slot] = exact_key(fabsf(wf), sc_);
                        }
                    }
                });
                __syncthreads();
                if (warp < nl && fl[warp].ok) bracket_rank(cand[warp], fl[warp], lane);
                __syncthreads();
            }
        }
        if (tid < COL_LINES && tid < nl && fl[tid].ok) st[tid].pending = 0u;
        __syncthreads();
        uint32_t pend = 0u;
#pragma unroll
        for (int j = 0; j < COL_LINES; ++j) pend |= (j < nl) ? st[j].pending : 0u;
        any_pending = pend != 0u;
    }

    Sched sc;
    sched_begin(sc, STAGE_ROUNDED, 31, 0);
    while (any_pending) {
        for (int i = tid; i < COL_LINES * COL_COPIES * HBINS; i += COL_THREADS) hist[i] = 0u;
        __syncthreads();
        uint32_t t32[COL_LINES];
#pragma unroll
        for (int j = 0; j < COL_LINES; ++j) t32[j] = (j < nl && st[j].pending) ? st[j].tau32 : 0xffffffffu;
        const int mode = count_mode(sc);
        if (mode == COUNT_ALL) count_pass(std::integral_constant<int, COUNT_ALL>{}, sc, t32);
        else if (mode == COUNT_ROUNDED) count_pass(std::integral_constant<int, COUNT_ROUNDED>{}, sc, t32);
        else count_pass(std::integral_constant<int, COUNT_TIED>{}, sc, t32);
        __syncthreads();
        if (warp < nl && st[warp].pending) bucket_step<COL_COPIES>(hist + warp * (COL_COPIES * HBINS), st[warp], sc, lane, &s_long);
        __syncthreads();
        uint32_t pending = 0u;
#pragma unroll
        for (int j = 0; j < COL_LINES; ++j) pending |= (j < nl) ? st[j].pending : 0u;
        if (!pending) break;
        const bool was_rounded = sc.stage == STAGE_ROUNDED;
        if (!sched_next<BF16>(sc, s_long != 0u, p.idx_bits)) break;
        if (was_rounded && s_long && tid < COL_LINES) st[tid].base = 0ull;   // read again only after the next barrier
    }
    if (tid < nl) {
        DASS_ST(&p.results[c0 + tid], fl[tid].ok ? fl[tid].res : line_result(st[tid], idx_top));
        if (p.cand_count) DASS_ST(&p.cand_count[c0 + tid], 0u);
    }
}

template <bool BF16, bool ALONG, bool TMA>
static cudaError_t launch_cols_as(const SelectParams &p, cudaStream_t st)
{
    CUtensorMap map;
    memset(&map, 0, sizeof(map));
    static_assert(COL_COPIES == 1, "the bracket sweep lays its histograms out with stride HSTRIDE");
    size_t smem = (size_t)COL_LINES * HSTRIDE * sizeof(uint32_t);
    if (TMA) {
        if (!tile_map_bf16(&map, p.W, p.rows, p.cols, p.ld, COL_LINES, SR_BOX_ROWS)) return cudaErrorInvalidValue;
        smem += 128 + SR_STAGES * SR_STAGE_BYTES + SR_STAGES * 8;
    }
    // the radix select lays its 2048-bin histograms over the same bytes (the bracket's bins and the ring are idle by then)
    const size_t radix_smem = (size_t)COL_LINES * COL_COPIES * HBINS * sizeof(uint32_t);
    smem = smem < radix_smem ? radix_smem : smem;
    cudaError_t e = cudaFuncSetAttribute(select_cols_kernel<BF16, ALONG, TMA>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    select_cols_kernel<BF16, ALONG, TMA><<<(unsigned)((p.cols + COL_LINES - 1) / COL_LINES), COL_THREADS, smem, st>>>(map, p);
    return cudaGetLastError();
}
template <bool BF16>
static cudaError_t launch_cols(const SelectParams &p, cudaStream_t st)
{
    // bulk copies need whole boxes of 8 columns x 256 rows inside the matrix, and the sweep they feed runs on long lines only
    const bool tma = BF16 && p.cols >= COL_LINES && p.L >= FAST_MIN_L && p.L <= FAST_MAX_L;
    if constexpr (BF16) {
        if (tma) return p.scale_along_line ? launch_cols_as<true, true, true>(p, st) : launch_cols_as<true, false, true>(p, st);
    }
    return p.scale_along_line ? launch_cols_as<BF16, true, false>(p, st) : launch_cols_as<BF16, false, false>(p, st);
}

cudaError_t select_launch_cols(const SelectParams &p, bool bf16, cudaStream_t st)
{
    return bf16 ? launch_cols<true>(p, st) : launch_cols<false>(p, st);
}

}  // namespace dass
