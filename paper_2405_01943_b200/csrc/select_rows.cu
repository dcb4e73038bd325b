// Unstructured selection, lines that are matrix rows (output-balanced: a row of Wd): the two-pass streaming kernel and
// the radix-select kernel that takes short lines and the rows the first one could not decide.
#include "select_common.cuh"

namespace dass {

// ---------------------------------------------------------------- lines that are matrix rows
// One CTA per row: the row is read once with 16-byte loads into shared memory, selected there and written out
// (mask bytes and the pruned copy) by the same CTA.
constexpr int ROW_THREADS = 256;
constexpr int ROW_COPIES = 1;                   // histogram copies the lanes spread over (2 measured slower: clearing and folding cost more than the conflicts)

template <bool BF16>
__global__ void __launch_bounds__(ROW_THREADS) select_rows_kernel(const SelectParams p)
{
    using elem_t = typename std::conditional<BF16, uint16_t, uint32_t>::type;
    constexpr int EPV = 16 / sizeof(elem_t);                     // elements per 16-byte vector
    extern __shared__ __align__(16) unsigned char u_smem[];
    elem_t *line_mem = reinterpret_cast<elem_t *>(u_smem);       // [lpad]
    uint32_t *hist = reinterpret_cast<uint32_t *>(u_smem + (size_t)p.lpad * sizeof(elem_t));   // [ROW_COPIES][HBINS]
    __shared__ Line st;
    __shared__ uint32_t s_long;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t nchunks = p.lpad >> 3;
    const uint32_t idx_top = (uint32_t)((1ull << p.idx_bits) - 1ull);
    // every row, or the rows the streaming kernel listed as undecided
    const int64_t n_lines = p.line_list ? (int64_t)DASS_LD(p.line_count) : p.rows;
    for (int64_t li = blockIdx.x; li < n_lines; li += gridDim.x) {
        const int64_t row = p.line_list ? (int64_t)DASS_LD(&p.line_list[li]) : li;
        const float line_scale = p.scale_along_line ? 0.0f : DASS_LD(&p.scale[row]);
        const elem_t *wrow = static_cast<const elem_t *>(p.W) + row * p.ld;
        const int64_t nfull = p.L >> 3;                  // chunks whose 8 elements all exist

        // ---------------------------------------------------------------- radix select on the line in shared memory
        {   // rows are 16-byte aligned and padded to whole vectors by the ld rule; what a vector drags in past L is
            // never used (every consumer checks the index against L)
            const uint4 *src = reinterpret_cast<const uint4 *>(wrow);
            uint4 *dst = reinterpret_cast<uint4 *>(line_mem);
            const int64_t nvec = (p.L + EPV - 1) / EPV;
            for (int64_t v = tid; v < (int64_t)(p.lpad / EPV); v += ROW_THREADS)
                dst[v] = v < nvec ? DASS_LD_CS(src + v) : make_uint4(0u, 0u, 0u, 0u);
        }
        if (tid == 0) { line_init(st, p.k); s_long = 0u; }

        // the 8 signed weights and scales of chunk q
        auto fetch = [&](int64_t q, float (&w)[8], float (&sc)[8]) {
            Chunk<BF16> ch;
            chunk_from<BF16>(ch, reinterpret_cast<const uint4 *>(line_mem + q * 8));
    #pragma unroll
            for (int j = 0; j < 8; ++j) w[j] = chunk_float<BF16>(ch, j);
            if (p.scale_along_line) {
                const float4 s0 = DASS_LD_G(reinterpret_cast<const float4 *>(p.scale + q * 8));
                const float4 s1 = DASS_LD_G(reinterpret_cast<const float4 *>(p.scale + q * 8) + 1);   // the vector is padded to 8
                sc[0] = s0.x; sc[1] = s0.y; sc[2] = s0.z; sc[3] = s0.w; sc[4] = s1.x; sc[5] = s1.y; sc[6] = s1.z; sc[7] = s1.w;
            } else {
    #pragma unroll
                for (int j = 0; j < 8; ++j) sc[j] = line_scale;
            }
        };
        uint32_t *my_hist = hist + (lane % ROW_COPIES) * HBINS;
        auto count_pass = [&](auto mode_tag, const Sched &sc, uint32_t t32) {
            constexpr int MODE = decltype(mode_tag)::value;
            for (int64_t q = tid; q < nfull; q += ROW_THREADS) {
                float w[8], s[8];
                fetch(q, w, s);
    #pragma unroll
                for (int j = 0; j < 8; ++j) count_element<MODE>(my_hist, st, t32, w[j], s[j], (uint32_t)(q * 8 + j), sc, idx_top);
            }
            if (tid == 0 && nfull < nchunks) {           // the ragged last chunk
                float w[8], s[8];
                fetch(nfull, w, s);
    #pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (nfull * 8 + j < p.L) count_element<MODE>(my_hist, st, t32, w[j], s[j], (uint32_t)(nfull * 8 + j), sc, idx_top);
            }
        };

        Sched sc;
        sched_begin(sc, STAGE_ROUNDED, 31, 0);
        for (;;) {
            for (int i = tid; i < ROW_COPIES * HBINS; i += ROW_THREADS) hist[i] = 0u;
            __syncthreads();
            const uint32_t t32 = st.tau32;
            const int mode = count_mode(sc);
            if (mode == COUNT_ALL) count_pass(std::integral_constant<int, COUNT_ALL>{}, sc, t32);
            else if (mode == COUNT_ROUNDED) count_pass(std::integral_constant<int, COUNT_ROUNDED>{}, sc, t32);
            else count_pass(std::integral_constant<int, COUNT_TIED>{}, sc, t32);
            __syncthreads();
            if (warp == 0) bucket_step<ROW_COPIES>(hist, st, sc, lane, &s_long);
            __syncthreads();
            if (!st.pending) break;
            const bool was_rounded = sc.stage == STAGE_ROUNDED;
            if (!sched_next<BF16>(sc, s_long != 0u, p.idx_bits)) break;
            if (was_rounded && s_long && tid == 0) st.base = 0ull;     // read again only after the next barrier
        }

        // ---------------------------------------------------------------- emit in place
        const LineResult res = line_result(st, idx_top);
        for (int64_t q = tid; q < nchunks; q += ROW_THREADS) {
            float a[8], s[8];
            fetch(q, a, s);
            uint32_t keep = 0u;
    #pragma unroll
            for (int j = 0; j < 8; ++j)
                if (q * 8 + j < p.L && keeps(res, a[j], s[j], q * 8 + j)) keep |= 1u << j;
            const int64_t e0 = q * 8;
            const int64_t left = p.L - e0;
            const int nvalid = left >= 8 ? 8 : (int)left;
            if (p.mask) DASS_ST(&reinterpret_cast<uint8_t *>(p.mask + row * p.wpr)[q], (uint8_t)keep);   // byte q = columns 8q..8q+7
            if (p.Wp) {
                Chunk<BF16> ch;
                chunk_from<BF16>(ch, reinterpret_cast<const uint4 *>(line_mem + e0));
                chunk_apply_mask<BF16>(ch, keep);
                chunk_store<BF16>(ch, p.Wp, row * p.ld + e0, nvalid);
            }
        }
        __syncthreads();                             // the next line reuses the shared memory
    }
}

// ---------------------------------------------------------------- lines that are matrix rows: two streaming passes
// One CTA per RS_ROWS adjacent rows and nothing cached: the first pass reads the rows and fills the histograms of
// their brackets, one warp per row finds the bin that holds the cut, and the second pass reads the rows again (from
// L2) and writes the outputs -- every element above that bin stays, every element below it goes, and the handful
// inside it are set aside, ranked by the row's warp at the end and patched into the outputs.  A row whose bracket
// misses, or whose bin holds too many elements, is put on a list for the radix kernel.  The rows of a CTA share every
// load of the scale vector, which is twice the bytes of a bf16 row and the largest user of the load/store pipe.
constexpr int RS_THREADS = 256;
constexpr int RS_ROWS = 2;
constexpr int RS_SAMPLE = SELECT_SAMPLE;        // evenly spaced elements of a row that place its bracket
constexpr int RS_HSTRIDE = BBINS + 32;          // a row's bins, then one idle word per lane (the sample's 256 + 256 counters fit in front)

// ALONG: the scale varies along the row (one per column) rather than being one number per row.
template <bool BF16, bool ALONG>
__global__ void __launch_bounds__(RS_THREADS, 4) select_rows_stream_kernel(const SelectParams p)
{
    using elem_t = typename std::conditional<BF16, uint16_t, uint32_t>::type;
    __shared__ uint32_t hist[RS_ROWS * RS_HSTRIDE];
    __shared__ uint32_t s_over[RS_ROWS];             // sample keys above the window
    __shared__ FastLine fl[RS_ROWS];
    __shared__ CandSet cand[RS_ROWS];
    __shared__ uint32_t cand_raw[RS_ROWS][CAND_CAP]; // the stored weights of the elements set aside

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t row0 = (int64_t)blockIdx.x * RS_ROWS;
    const int nr = (int)(p.rows - row0 < RS_ROWS ? p.rows - row0 : RS_ROWS);     // rows of this CTA
    const int64_t nchunks = p.lpad >> 3;
    const int64_t nfull = p.L >> 3;                  // chunks whose 8 elements all exist
    const uint32_t hist_s = smem_u32(hist);
    float line_scale[RS_ROWS];
    const elem_t *wrow[RS_ROWS];
#pragma unroll
    for (int r = 0; r < RS_ROWS; ++r) {
        const int64_t row = row0 + (r < nr ? r : 0);                 // a missing row repeats the first (its results are dropped)
        wrow[r] = static_cast<const elem_t *>(p.W) + row * p.ld;
        line_scale[r] = ALONG ? 0.0f : DASS_LD(&p.scale[row]);
    }

    // chunk q (8 columns) of every row as stored, and the scales of its columns
    auto load_chunk = [&](int64_t q, Chunk<BF16> (&ch)[RS_ROWS], float (&sc)[8]) {
#pragma unroll
        for (int r = 0; r < RS_ROWS; ++r) {
            const uint4 *src = reinterpret_cast<const uint4 *>(wrow[r] + q * 8);
            const uint4 v0 = DASS_LD_G(src);
            ch[r].w[0] = v0.x; ch[r].w[1] = v0.y; ch[r].w[2] = v0.z; ch[r].w[3] = v0.w;
            if constexpr (!BF16) {
                const uint4 v1 = DASS_LD_G(src + 1);         // a row's pitch covers whole 8-element chunks
                ch[r].w[4] = v1.x; ch[r].w[5] = v1.y; ch[r].w[6] = v1.z; ch[r].w[7] = v1.w;
            }
        }
        if constexpr (ALONG) {
            const float4 s0 = DASS_LD_G(reinterpret_cast<const float4 *>(p.scale + q * 8));
            const float4 s1 = DASS_LD_G(reinterpret_cast<const float4 *>(p.scale + q * 8) + 1);   // the vector is padded to 8
            sc[0] = s0.x; sc[1] = s0.y; sc[2] = s0.z; sc[3] = s0.w; sc[4] = s1.x; sc[5] = s1.y; sc[6] = s1.z; sc[7] = s1.w;
        }
    };
    // the 8 keys of a row's chunk: bits of fl32(|w| * scale)
    auto keys_of = [&](int r, const Chunk<BF16> &ch, const float (&sc)[8], uint32_t (&key)[8]) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float sv = ALONG ? sc[j] : line_scale[r];
            if constexpr (BF16) key[j] = __float_as_uint((j & 1) ? prod_hi(ch.w[j >> 1], sv) : prod_lo(ch.w[j >> 1], sv));
            else key[j] = __float_as_uint(fabsf(__uint_as_float(ch.w[j])) * sv);
        }
    };
    // runs f(q, chunks of all rows, scales, valid elements) over the rows
    auto sweep = [&](auto &&f) {
        int64_t q = tid;
        for (; q < nfull; q += RS_THREADS) {
            Chunk<BF16> ch[RS_ROWS];
            float sc[8];
            load_chunk(q, ch, sc);
            f(q, ch, sc, 8);
        }
        if (q < nchunks) {                           // the ragged last chunk (one thread)
            Chunk<BF16> ch[RS_ROWS];
            float sc[8];
            load_chunk(q, ch, sc);
            f(q, ch, sc, (int)(p.L - q * 8));
        }
    };

    // ---------------------------------------------------------------- the brackets, from a sample of each row
    constexpr int PER_THREAD = RS_SAMPLE / RS_THREADS;
    uint32_t skey[RS_ROWS][PER_THREAD];
    // per row, in its histogram's space: 256 exponent counts, then FINE_BINS fine bins
    for (int i = tid; i < RS_ROWS * RS_HSTRIDE; i += RS_THREADS) hist[i] = 0u;
    if (tid < RS_ROWS) { fl[tid].ok = 0u; s_over[tid] = 0u; }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < PER_THREAD; ++u) {
        const int64_t e = ((int64_t)(tid + u * RS_THREADS) * p.L) / RS_SAMPLE;
        float sv = 0.0f;
        if constexpr (ALONG) sv = DASS_LD_G(p.scale + e);
#pragma unroll
        for (int r = 0; r < RS_ROWS; ++r) {
            float wf;
            if constexpr (BF16) wf = __uint_as_float((uint32_t)DASS_LD_G(wrow[r] + e) << 16);
            else wf = __uint_as_float(DASS_LD_G(wrow[r] + e));
            skey[r][u] = product_key(wf, ALONG ? sv : line_scale[r]);
        }
    }
#pragma unroll
    for (int r = 0; r < RS_ROWS; ++r) {
#pragma unroll
        for (int u = 0; u < PER_THREAD; ++u) {
            // a warp's keys share a few exponents: one update per distinct exponent
            const uint32_t e = skey[r][u] >> 23;
            const uint32_t same = __match_any_sync(FULL_MASK, e);
            if (lane == __ffs((int)same) - 1) atomicAdd(hist + r * RS_HSTRIDE + e, (uint32_t)__popc(same));
        }
    }
    __syncthreads();
    const int target = (int)win_target(p.k, p.L, RS_SAMPLE);
    if (warp < nr) window_from_exponents(hist + warp * RS_HSTRIDE, fl[warp], (uint32_t)target, lane);
    __syncthreads();
#pragma unroll
    for (int r = 0; r < RS_ROWS; ++r) {
        const uint32_t wlo = fl[r < nr ? r : 0].lo;
#pragma unroll
        for (int u = 0; u < PER_THREAD; ++u) {
            const uint32_t off = skey[r][u] - wlo;
            if (off < WIN_SPAN) atomicAdd(hist + r * RS_HSTRIDE + 256 + (off >> FINE_SHIFT), 1u);
            else if (skey[r][u] > wlo) atomicAdd(&s_over[r], 1u);
        }
    }
    __syncthreads();
    if (warp < nr) bracket_from_fine(hist + warp * RS_HSTRIDE + 256, s_over[warp], fl[warp], target, p.margin, lane);
    __syncthreads();
    for (int i = tid; i < RS_ROWS * RS_HSTRIDE; i += RS_THREADS) hist[i] = 0u;
    __syncthreads();

    // ---------------------------------------------------------------- first pass: histograms of the brackets
    {   // every lane updates a counter: its element's bin inside the bracket (which spans all BBINS bins), else a word of
        // its own behind the bins that nobody reads; the elements below the bracket are counted, those above it follow
        // from the line's length
        uint32_t lo[RS_ROWS], mul[RS_ROWS], below[RS_ROWS];
#pragma unroll
        for (int r = 0; r < RS_ROWS; ++r) { lo[r] = fl[r < nr ? r : 0].lo; mul[r] = fl[r < nr ? r : 0].mul; below[r] = 0u; }
        const uint32_t idle_bin = (uint32_t)(BBINS + lane);
        sweep([&](int64_t, const Chunk<BF16> (&ch)[RS_ROWS], const float (&sc)[8], int nvalid) {
#pragma unroll
            for (int r = 0; r < RS_ROWS; ++r) {
                uint32_t key[8];
                keys_of(r, ch[r], sc, key);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (j < nvalid) {
                        const uint32_t off = key[j] - lo[r];         // keys are below 2^31: the top bit says "below lo"
                        asm volatile("red.shared.add.u32 [%0], 1;"
                                     ::"r"(hist_s + (uint32_t)(r * RS_HSTRIDE * 4) + (min(__umulhi(off, mul[r]), idle_bin) << 2)) : "memory");
                        below[r] = __umulhi(off, 2u) + below[r];
                    }
                }
            }
        });
#pragma unroll
        for (int r = 0; r < RS_ROWS; ++r) {
            uint32_t a = below[r];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(FULL_MASK, a, off);
            if (lane == 0 && a && r < nr) atomicAdd(&fl[r].below, a);
        }
    }
    __syncthreads();
    if (warp < nr) bracket_pick_bin(hist + warp * RS_HSTRIDE, fl[warp], p.k, lane, p.L);
    __syncthreads();
    bool live[RS_ROWS];                              // the same for every thread
    bool any_live = false;
#pragma unroll
    for (int r = 0; r < RS_ROWS; ++r) { live[r] = r < nr && fl[r].ok != 0u; any_live |= live[r]; }
    if (tid < nr && !fl[tid].ok)                     // left to the radix kernel
        DASS_ST(&p.line_list[atomicAdd(p.line_count, 1u)], (uint32_t)(row0 + tid));
    if (!any_live) return;

    // ---------------------------------------------------------------- second pass: outputs, the cut's bin set aside
    {
        uint32_t blo[RS_ROWS], bhi[RS_ROWS], bw[RS_ROWS];
#pragma unroll
        for (int r = 0; r < RS_ROWS; ++r) { blo[r] = fl[r < nr ? r : 0].blo; bhi[r] = fl[r < nr ? r : 0].bhi; bw[r] = bhi[r] - blo[r]; }
        sweep([&](int64_t q, Chunk<BF16> (&ch)[RS_ROWS], const float (&sc)[8], int nvalid) {
#pragma unroll
            for (int r = 0; r < RS_ROWS; ++r) {
                if (!live[r]) continue;
                const int64_t row = row0 + r;
                uint32_t key[8];
                keys_of(r, ch[r], sc, key);
                bool some = false;                   // an element of this chunk lies in the cut's bin
#pragma unroll
                for (int j = 0; j < 8; ++j) some |= j < nvalid && key[j] - blo[r] < bw[r];
                if (some) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (j < nvalid && key[j] - blo[r] < bw[r]) {
                            const uint32_t slot = atomicAdd(&fl[r].ncoll, 1u);
                            if (slot < (uint32_t)CAND_CAP) {
                                const float wf = chunk_float<BF16>(ch[r], j);
                                cand[r].key[slot] = key[j]; cand[r].idx[slot] = (uint32_t)(q * 8 + j);
                                cand[r].k64[slot] = exact_key(fabsf(wf), ALONG ? sc[j] : line_scale[r]);
                                cand_raw[r][slot] = __float_as_uint(wf);
                            }
                        }
                    }
                }
                // below bhi: pruned here (the bin's survivors come back at the end)
                uint32_t keep = 0u;
                if constexpr (BF16) {
                    uint32_t z[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        z[k] = pn_prmt(key[2 * k] - bhi[r], key[2 * k + 1] - bhi[r], 0xFFBBu);   // keys are below 2^31: the sign is the order
                        ch[r].w[k] &= ~z[k];
                    }
                    // lane masks to bits: even columns sit in the low lanes, odd ones 16 bits up
                    const uint32_t x = (z[0] & 0x00020001u) | (z[1] & 0x00080004u) | (z[2] & 0x00200010u) | (z[3] & 0x00800040u);
                    keep = ~(x | (x >> 16)) & 0xffu;
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t z = (uint32_t)((int32_t)(key[j] - bhi[r]) >> 31);
                        ch[r].w[j] &= ~z;
                        keep |= ~z & (1u << j);
                    }
                }
                keep &= (1u << nvalid) - 1u;
                if (p.mask) DASS_ST(&reinterpret_cast<uint8_t *>(p.mask + row * p.wpr)[q], (uint8_t)keep);   // byte q = columns 8q..8q+7
                if (p.Wp) chunk_store<BF16>(ch[r], p.Wp, row * p.ld + q * 8, nvalid);
            }
        });
    }
    __syncthreads();

    // ---------------------------------------------------------------- the cut's bin: ranked, survivors patched in
    bool my_row_live = false;                        // warp r ranks row r
#pragma unroll
    for (int r = 0; r < RS_ROWS; ++r) my_row_live |= warp == r && live[r];
    if (my_row_live) {
        const int r = warp;
        const int64_t row = row0 + r;
        bracket_rank(cand[r], fl[r], lane);
        __syncwarp();
        if (fl[r].ok) {                              // always: the bin's count was checked and the keys are distinct
            const LineResult res = fl[r].res;
            const int n = (int)fl[r].ncoll;
            for (int i = lane; i < n; i += 32) {
                const uint32_t key = cand[r].key[i], idx = cand[r].idx[i];
                const unsigned long long k64 = cand[r].k64[i];
                const bool stays = key > res.tau32 ||
                                   (key == res.tau32 && (!res.exact || k64 > res.tau64 || (k64 == res.tau64 && (long long)idx <= res.cut)));
                if (stays) {
                    if (p.mask) atomicOr(p.mask + row * p.wpr + (idx >> 5), 1u << (idx & 31u));
                    if (p.Wp) {
                        if constexpr (BF16) DASS_ST(static_cast<uint16_t *>(p.Wp) + row * p.ld + idx, (uint16_t)(cand_raw[r][i] >> 16));
                        else DASS_ST(static_cast<uint32_t *>(p.Wp) + row * p.ld + idx, cand_raw[r][i]);
                    }
                }
            }
        } else if (lane == 0 && p.status) {
            atomicMax(p.status, (int)DASS_ERR_INTERNAL);
        }
    }
}

// Dynamic shared memory of the row-line kernel: the cached line and one histogram.
size_t select_row_smem_bytes(int64_t L, bool bf16)
{
    const int64_t lpad = (L + 7) / 8 * 8;
    return (size_t)lpad * (bf16 ? 2 : 4) + (size_t)ROW_COPIES * HBINS * sizeof(uint32_t);
}

template <bool BF16>
static cudaError_t launch_rows(SelectParams p, uint32_t *line_count, uint32_t *line_list, cudaStream_t st)
{
    const size_t smem = select_row_smem_bytes(p.L, BF16);
    cudaError_t e = cudaFuncSetAttribute(select_rows_kernel<BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (p.L < FAST_MIN_L || p.L > FAST_MAX_L) {      // short or very long lines: the radix kernel alone, one CTA per row
        p.line_count = nullptr; p.line_list = nullptr;
        select_rows_kernel<BF16><<<(unsigned)p.rows, ROW_THREADS, smem, st>>>(p);
        return cudaGetLastError();
    }
    // the streaming kernel decides the rows it can and lists the others; the radix kernel works the list off
    p.line_count = line_count; p.line_list = line_list;
    e = cudaMemsetAsync(line_count, 0, sizeof(uint32_t), st);
    if (e != cudaSuccess) return e;
    const unsigned stream_grid = (unsigned)((p.rows + RS_ROWS - 1) / RS_ROWS);
    if (p.scale_along_line) select_rows_stream_kernel<BF16, true><<<stream_grid, RS_THREADS, 0, st>>>(p);
    else select_rows_stream_kernel<BF16, false><<<stream_grid, RS_THREADS, 0, st>>>(p);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    int per_sm = 1;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, select_rows_kernel<BF16>, ROW_THREADS, smem);
    if (e != cudaSuccess) return e;
    const int64_t resident = (int64_t)device_sm_count() * (per_sm > 0 ? per_sm : 1);
    select_rows_kernel<BF16><<<(unsigned)(p.rows < resident ? p.rows : resident), ROW_THREADS, smem, st>>>(p);
    return cudaGetLastError();
}

cudaError_t select_launch_rows(const SelectParams &p, bool bf16, uint32_t *line_count, uint32_t *line_list, cudaStream_t st)
{
    return bf16 ? launch_rows<true>(p, line_count, line_list, st) : launch_rows<false>(p, line_count, line_list, st);
}

}  // namespace dass
