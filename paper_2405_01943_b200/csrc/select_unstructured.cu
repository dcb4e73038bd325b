// Unstructured DaSS selection at a sparsity ratio s (Section 3, "Pruning Granularity"): in every comparison
// line -- a column of Wg / Wu (all neurons at one input: input-balanced) or a row of Wd (output-balanced) --
// the floor(s * L) weights with the lowest Eq. 4 / Eq. 5 score are pruned.  No sort.
//
// The order of the oracle, "higher score first, lower index first", is the order of a three-part key: the
// rounded product fl32(|w| * scale), then the exact double product, then the index counted from the top.
//
// Lines of FAST_MIN_L elements and more are decided by two streaming sweeps: 1024 evenly spaced elements of the line
// give, through two small histograms (no sort), a bracket of rounded products that holds the cut unless the sample is
// four standard deviations off; the first sweep reduces every element into a 2048-bin histogram of the bracket (those
// outside land on idle words) and counts the elements below it; one warp finds the bin that holds the cut; the second
// sweep writes the outputs -- above the bin stays, below it goes -- and sets the bin's few elements aside; one warp
// ranks those by the full key and puts the survivors back.  A line whose bracket misses, or whose bin holds more than
// CAND_CAP elements, is decided by the radix select: the k-th largest key is found 11 bits at a time with
// shared-memory histograms, and a line stops as soon as the bucket at the cut holds exactly the survivors still
// wanted (exact products and indices are consulted only where rounded products tie across the cut).
//
// Lines that are matrix rows: select_rows_stream_kernel (both sweeps, two rows per CTA), then select_rows_kernel
// (radix select, the row cached in shared memory) for the rows the first kernel listed, or for every row when the
// lines are short.  Lines that are matrix columns: select_cols_kernel (one CTA per strip of 8 adjacent columns: sample,
// first sweep, bin; radix select inside the kernel where needed) publishes a LineResult per column, a streaming
// kernel with coalesced rows emits (select_emit_stream_kernel for bf16, select_emit_cols_kernel for f32), and
// select_fix_cols_kernel ranks what the emit pass set aside.
#include <cmath>
#include <cstring>
#include <type_traits>

#include "stream_units.cuh"

namespace dass {

// f(integral_constant<int, 0>) ... f(integral_constant<int, N - 1>)
template <int N, typename F>
__device__ __forceinline__ void static_for(F &&f)
{
    if constexpr (N > 0) {
        static_for<N - 1>(f);
        f(std::integral_constant<int, N - 1>{});
    }
}

// What the selection found for one line; enough to decide every element of the line locally:
// keep iff p > tau32, or p == tau32 and (not exact, or k64 > tau64, or k64 == tau64 and index <= cut).
struct LineResult {
    unsigned long long tau64;
    long long cut;
    uint32_t tau32;
    uint32_t exact;      // 0 / 1 as above; LINE_BIN: the line is decided up to one histogram bin, see below
};
// A column whose cut is known up to a bin [blo, bhi) of rounded products: every element at or above bhi stays,
// every element below blo goes, and of the `bucket` elements inside the bin the krem2 largest stay.  The emit pass
// sets those elements aside in per-column lists and a last small kernel ranks them.  Stored in a LineResult as
// tau32 = bhi, exact = LINE_BIN, tau64 = blo | krem2 << 32, cut = bucket.
constexpr uint32_t LINE_BIN = 2u;
struct CandLists {               // per column: how many elements were set aside, and CAND_CAP slots of each array
    uint32_t *count;
    uint32_t *key;               // rounded product
    uint32_t *idx;               // row
    uint32_t *raw;               // the stored weight, in the upper 16 bits for bf16
};

struct SelectParams {
    const void *W;
    void *Wp;            // nullable (row lines only: the kernel emits)
    uint32_t *mask;      // nullable (row lines only)
    const float *scale;  // precomputed fl32(norm^alpha), padded with zeros to a multiple of 8
    struct LineResult *results;   // per-column thresholds (column lines only: a second, streaming kernel emits)
    int64_t rows, cols, ld;
    int64_t wpr;         // mask words per matrix row
    int64_t L;           // line length
    int64_t lpad;        // L rounded up to 8
    uint32_t k;          // survivors per line
    int idx_bits;        // bits of L - 1 (at least 1): width of the index part of the key
    int scale_along_line;   // 1: scale[e] varies along the line; 0: scale[line]
    int margin;             // sampled bracket: sample positions on either side of the wanted rank (four standard deviations)
    uint32_t *line_count;   // row lines: how many lines the streaming kernel left undecided, and which
    uint32_t *line_list;    // (both null: the radix kernel takes every row)
    uint32_t *cand_count;   // column lines, bf16: per-column count of the elements the emit pass sets aside (cleared here)
    int *status;            // device status word for bounded waits that ran out
};

// out[i] = fl32(norm[i]^alpha) for i < n, 0 for the padding up to npad (a multiple of 8, so that the selection
// kernel can read whole 8-element chunks)
__global__ void scale_vector_kernel(const float *__restrict__ norm, int64_t n, int64_t npad, int mode, float alpha,
                                    float *__restrict__ out)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) DASS_ST(&out[i], scale_from_norm(DASS_LD(&norm[i]), mode, alpha));
    else if (i < npad) DASS_ST(&out[i], 0.0f);
}

// ---------------------------------------------------------------- radix select on a three-part key
// The order "higher score first, lower index first" is the order of the key (p, r, ~index), compared part by
// part: p = bits of fl32(|w| * scale) (rounding is monotone, so p decides every pair whose rounded products
// differ), r = bits of the exact double product minus a per-line base (decides pairs whose rounded products are
// equal), and the index counted down from the top (lower index first).  The k-th largest key of a line is found
// digit by digit, 11 bits per pass, with a shared-memory histogram of 2048 bins per line.  A line is decided as
// soon as the bucket that holds the k-th key holds exactly as many candidates as are still to be kept: all of
// them stay, and "key >= chosen prefix" is the rule; most lines end inside p, after two or three passes.
constexpr int HB = 11;                          // bits per digit
constexpr int HBINS = 1 << HB;

enum : int { STAGE_ROUNDED = 0, STAGE_EXACT = 1, STAGE_INDEX = 2 };

struct Line {                    // selection state of one comparison line (shared memory)
    unsigned long long tau64;    // digits chosen so far of r = (bits of the exact product) - base
    unsigned long long base;
    uint32_t tau32;              // digits chosen so far of p
    uint32_t tauidx;             // digits chosen so far of (idx_top - index)
    uint32_t krem;               // survivors still to be taken among the current candidates
    uint32_t pending;            // 1 until the line is decided
    uint32_t done_stage;         // part of the key in which it was decided
    uint32_t pad_;
};

// The digit being counted: bits [shift, shift + bits) of the current part of the key.  A part ends when its
// digits reach bit `stop` (the bits below are known to be zero) or bit 0.
struct Sched { int stage, shift, bits, stop; };

__device__ __forceinline__ void sched_begin(Sched &s, int stage, int key_bits, int stop)
{
    s.stage = stage;
    s.bits = key_bits < HB ? key_bits : HB;
    s.shift = key_bits - s.bits;
    s.stop = stop;
}

// Moves to the next digit; false when the whole key has been used (cannot happen while a line is pending: the
// index part makes all keys distinct).  `long_exact`: some line's threshold product is a float denormal, where the
// distance between neighbouring floats is not 2^29 doubles: r is then the whole 63-bit pattern (base 0).
template <bool BF16>
__device__ __forceinline__ bool sched_next(Sched &s, bool long_exact, int idx_bits)
{
    if (s.shift > 0 && s.shift > s.stop) {
        const int b = s.shift < HB ? s.shift : HB;
        s.shift -= b;
        s.bits = b;
        return true;
    }
    if (s.stage == STAGE_ROUNDED) {
        // equal rounded products: the exact products lie within half a float ulp = 2^28 doubles of the threshold,
        // so r < 2^30; a bf16 x float product has at most 32 significant bits: the low 21 bits of r are zero
        if (long_exact) sched_begin(s, STAGE_EXACT, 63, 0);
        else sched_begin(s, STAGE_EXACT, 30, BF16 ? 21 : 0);
        return true;
    }
    if (s.stage == STAGE_EXACT) { sched_begin(s, STAGE_INDEX, idx_bits, 0); return true; }
    return false;
}

__device__ __forceinline__ unsigned long long exact_key(float a, float s)
{
    return (unsigned long long)__double_as_longlong((double)a * (double)s);   // exact: at most 48 significant bits
}

__device__ __forceinline__ uint32_t bit_field(uint32_t v, int pos, int len)
{
    uint32_t d;
    asm("bfe.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(v), "r"(pos), "r"(len));
    return d;
}

// Element j of a chunk widened to float with its sign (exact for both types).
template <bool BF16>
__device__ __forceinline__ float chunk_float(const Chunk<BF16> &c, int j)
{
    if constexpr (BF16) return __uint_as_float((j & 1) ? (c.w[j >> 1] & 0xffff0000u) : (c.w[j >> 1] << 16));
    else return __uint_as_float(c.w[j]);
}

// How a pass treats an element: COUNT_ALL (first digit of p: every element is a candidate), COUNT_ROUNDED (later
// digits of p: candidates agree with the digits chosen so far), COUNT_TIED (exact and index parts: candidates
// have the threshold's rounded product).
enum : int { COUNT_ALL = 0, COUNT_ROUNDED = 1, COUNT_TIED = 2 };

// Counts one element (signed weight wf, scale s >= 0) of a line in the current pass.  The sign of the product is
// the weight's and sits in bit 31, which no digit and no comparison below looks at.  t32 = the line's tau32, or
// 0xffffffff when the line is decided (then only a non-finite product could match; its count is never read).
template <int MODE>
__device__ __forceinline__ void count_element(uint32_t *h, const Line &ln, uint32_t t32, float wf, float s, uint32_t idx,
                                              const Sched &sc, uint32_t idx_top)
{
    const uint32_t pk = __float_as_uint(__fmul_rn(wf, s));
    if (MODE == COUNT_ALL) {
        atomicAdd(h + bit_field(pk, sc.shift, sc.bits), 1u);
    } else if (MODE == COUNT_ROUNDED) {
        const uint32_t known = (~0u << (sc.shift + sc.bits)) & 0x7fffffffu;      // shift + bits <= 31
        if (((pk ^ t32) & known) == 0u) atomicAdd(h + bit_field(pk, sc.shift, sc.bits), 1u);
    } else if (((pk ^ t32) << 1) == 0u) {
        const unsigned long long r = exact_key(fabsf(wf), s) - ln.base;
        if (sc.stage == STAGE_EXACT) {
            const unsigned long long known = ~0ull << (sc.shift + sc.bits);       // shift + bits <= 63
            if (((r ^ ln.tau64) & known) == 0ull) atomicAdd(h + bit_field((uint32_t)(r >> sc.shift), 0, sc.bits), 1u);
        } else if (r == ln.tau64) {
            const uint32_t ik = idx_top - idx;
            const uint32_t known = ~0u << (sc.shift + sc.bits);                   // shift + bits <= 31
            if (((ik ^ ln.tauidx) & known) == 0u) atomicAdd(h + bit_field(ik, sc.shift, sc.bits), 1u);
        }
    }
}

__device__ __forceinline__ int count_mode(const Sched &sc)
{
    if (sc.stage != STAGE_ROUNDED) return COUNT_TIED;
    return sc.shift + sc.bits == 31 ? COUNT_ALL : COUNT_ROUNDED;
}

// One warp, one pending line: finds the bin that holds the krem-th largest candidate, appends its digit to the
// line's threshold and decides the line when the bin holds exactly the candidates still to be taken.
template <int COPIES>
__device__ __forceinline__ void bucket_step(uint32_t *h, Line &ln, const Sched &sc, int lane, uint32_t *s_long)
{
    uint32_t *mine_bins = h + lane * 64;              // this lane's 64 bins (of copy 0)
    uint32_t lane_sum = 0u;
#pragma unroll 4
    for (int i = 0; i < 64; ++i) {
        const int b = (i + lane) & 63;                // rotated start: the 32 lanes hit 32 banks
        uint32_t c = mine_bins[b];
        if (COPIES > 1) {                             // fold the copies into copy 0
#pragma unroll
            for (int r = 1; r < COPIES; ++r) c += mine_bins[r * HBINS + b];
            mine_bins[b] = c;
        }
        lane_sum += c;
    }
    uint32_t v = lane_sum;                            // becomes the sum over lanes >= this one
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t t = __shfl_down_sync(FULL_MASK, v, off);
        if (lane + off < 32) v += t;
    }
    const uint32_t krem = ln.krem;
    uint32_t above = v - lane_sum;                    // candidates in bins above this lane's
    const bool mine = above < krem && krem <= above + lane_sum;
    uint32_t d = 0u, g = 0u, bc = 0u;
    if (mine) {
        for (int i = 63; i >= 0; --i) {
            const uint32_t c = mine_bins[i];
            if (krem <= above + c) { d = (uint32_t)(lane * 64 + i); g = above; bc = c; break; }
            above += c;
        }
    }
    const uint32_t who = __ballot_sync(FULL_MASK, mine);
    const int src = who ? __ffs(who) - 1 : 0;
    const uint32_t digit = __shfl_sync(FULL_MASK, d, src);
    const uint32_t greater = __shfl_sync(FULL_MASK, g, src);
    const uint32_t bucket = __shfl_sync(FULL_MASK, bc, src);
    if (lane == 0) {
        const uint32_t left = krem - greater;
        ln.krem = left;
        if (sc.stage == STAGE_ROUNDED) ln.tau32 |= digit << sc.shift;
        else if (sc.stage == STAGE_EXACT) ln.tau64 |= (unsigned long long)digit << sc.shift;
        else ln.tauidx |= digit << sc.shift;
        if (bucket == left) {
            ln.pending = 0u;
            ln.done_stage = (uint32_t)sc.stage;
        } else if (sc.stage == STAGE_ROUNDED && sc.shift == 0) {
            // the rounded products tie across the cut: the exact part of the key goes on
            const uint32_t t = ln.tau32;
            if (t >= 0x00800000u) {
                ln.base = (unsigned long long)__double_as_longlong((double)__uint_as_float(t)) - (1ull << 28);
            } else {
                ln.base = 0ull;
                atomicOr(s_long, 1u);
            }
        }
    }
}

// What the emit step needs of a decided line.
__device__ __forceinline__ LineResult line_result(const Line &ln, uint32_t idx_top)
{
    LineResult r;
    r.tau32 = ln.tau32;
    r.exact = ln.done_stage != STAGE_ROUNDED ? 1u : 0u;
    r.tau64 = ln.base + ln.tau64;
    r.cut = ln.done_stage == STAGE_INDEX ? (long long)(idx_top - ln.tauidx) : 0x7fffffffffffffffll;
    return r;
}

__device__ __forceinline__ void line_init(Line &ln, uint32_t k)
{
    ln.tau64 = 0ull; ln.base = 0ull; ln.tau32 = 0u; ln.tauidx = 0u; ln.krem = k; ln.pending = 1u;
    ln.done_stage = STAGE_ROUNDED; ln.pad_ = 0u;
}

template <bool BF16>
__device__ __forceinline__ void chunk_from(Chunk<BF16> &c, const uint4 *src)    // shared or global, 16-byte aligned
{
    const uint4 a = src[0];
    c.w[0] = a.x; c.w[1] = a.y; c.w[2] = a.z; c.w[3] = a.w;
    if constexpr (!BF16) {
        const uint4 b = src[1];
        c.w[4] = b.x; c.w[5] = b.y; c.w[6] = b.z; c.w[7] = b.w;
    }
}

// keep bit of one element (signed weight a, scale s >= 0) under a decided line's rule
__device__ __forceinline__ bool keeps(const LineResult &res, float a, float s, long long idx)
{
    const uint32_t key = __float_as_uint(__fmul_rn(a, s)) & 0x7fffffffu;
    if (key != res.tau32) return key > res.tau32;
    if (!res.exact) return true;
    const unsigned long long k64 = exact_key(fabsf(a), s);
    return k64 > res.tau64 || (k64 == res.tau64 && idx <= res.cut);
}

// ---------------------------------------------------------------- sampled bracket in front of the radix select
constexpr int WIN_BELOW = 3;                    // the window: 3 octaves below the octave of the sample's quantile, that octave, 4 above
constexpr uint32_t WIN_SPAN = 1u << 26;         // 8 octaves of keys
constexpr int CAND_CAP = 160;                   // elements of the cut's bin that the final ranking takes (equal scales: ~100 equal bf16 magnitudes)
constexpr int64_t FAST_MIN_L = 4096;            // shorter lines go straight to the radix select

struct FastLine {                // bracket state of one comparison line (shared memory)
    uint32_t lo, hi;             // candidates: lo <= key < hi (key = bits of the rounded product, sign cleared)
    uint32_t blo, bhi;           // the bin of the bracket that holds the cut
    uint32_t mul;                // bin = floor((key - lo) * mul / 2^32): bins of an odd width, so that keys a power of two apart
                                 // (equal scales: bf16 magnitudes) spread over the shared-memory banks
    uint32_t above;              // elements with key >= hi
    uint32_t below;              // elements with key < lo (streaming kernels: above = L - below - inside)
    uint32_t krem2;              // rank, from the top and 1-based, of the last survivor inside [blo, bhi)
    uint32_t ncoll;              // elements collected from that bin
    uint32_t bucket;             // elements the histogram saw in that bin
    uint32_t ok;                 // the bracket still holds for this line
    LineResult res;
};

struct CandSet {                 // the collected elements of one line
    unsigned long long k64[CAND_CAP];
    uint32_t key[CAND_CAP];
    uint32_t idx[CAND_CAP];
};

__device__ __forceinline__ uint32_t product_key(float wf, float s) { return __float_as_uint(__fmul_rn(wf, s)) & 0x7fffffffu; }

// One warp: places the window of one line from the exponent histogram (256 bins, key >> 23) of its sample.  The
// octave that holds the sample's `target`-th largest key is found, and the window starts WIN_BELOW octaves below it.
// The line's true cut lies within a fraction of an octave of the sample's; if it does not lie in the window after
// all, bracket_pick_bin sees that from the counts and the line takes the radix select.
__device__ __forceinline__ void window_from_exponents(const uint32_t *eh, FastLine &f, uint32_t target, int lane)
{
    uint32_t c[8], mine = 0u;
#pragma unroll
    for (int i = 0; i < 8; ++i) { c[i] = eh[lane * 8 + i]; mine += c[i]; }
    uint32_t v = mine;                                // becomes the sum over lanes >= this one
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t t = __shfl_down_sync(FULL_MASK, v, off);
        if (lane + off < 32) v += t;
    }
    uint32_t above = v - mine;
    const bool here = above < target && target <= above + mine;
    int e = 0;
    if (here) {
#pragma unroll
        for (int i = 7; i >= 0; --i) {
            if (target <= above + c[i]) { e = lane * 8 + i; break; }
            above += c[i];
        }
    }
    const uint32_t who = __ballot_sync(FULL_MASK, here);
    e = who ? __shfl_sync(FULL_MASK, e, __ffs(who) - 1) : 0;
    if (lane == 0) {
        const int e0 = e > WIN_BELOW ? e - WIN_BELOW : 0;
        f.lo = (uint32_t)e0 << 23;
        f.hi = f.lo + WIN_SPAN;
        f.mul = 0u;
        f.above = 0u; f.below = 0u; f.ncoll = 0u; f.ok = 1u; f.krem2 = 0u; f.bucket = 0u; f.blo = 0u; f.bhi = 0u;
    }
}

// Rank, from the top, of the key that stands for the line's k-th largest in a sample of S.
__device__ __forceinline__ uint32_t win_target(uint32_t k, int64_t L, int S)
{
    const int64_t t = ((int64_t)k * S + L - 1) / L;
    return (uint32_t)(t < 1 ? 1 : (t > S ? S : t));
}

// One warp: narrows a line's window to a bracket [lo, hi) from the fine histogram of a larger sample (FINE_BINS bins
// of 2^FINE_SHIFT keys from the window's start; n_over = sample keys above the window).  With the sample sorted from
// the top, the line's cut lies between the sample's (t - m)-th and (t + m)-th key unless the sample is m positions
// off the expected rank (m is four standard deviations of that rank, set by the host); the bracket is those two
// keys' fine bins and what lies between.  About 2m/S of the line plus two fine bins falls inside; everything else
// is only counted.  A miss shows in bracket_pick_bin's counts and sends the line to the radix select.
// Bins of the bracket's histogram: BBINS of them (about a sixth of a line falls inside the bracket: 9 elements per bin
// for a line of 28672, and equal bf16 magnitudes lie 2^16 keys apart, many bin widths), bin = floor(offset * mul / 2^32)
// with mul = floor(2^32 / width), width odd and wide enough for BBINS bins to cover `span`.  Bin d holds the offsets
// [bin_start(d), bin_start(d + 1)).
constexpr int BBINS = 1024;
constexpr int64_t FAST_MAX_L = 1 << 18;         // longer lines would crowd the bins: radix select
__device__ __forceinline__ uint32_t bin_multiplier(uint32_t span)
{
    const uint32_t width = ((span + (uint32_t)BBINS - 1u) / (uint32_t)BBINS) | 1u;
    return (uint32_t)(0x100000000ull / (width < 3u ? 3u : width));
}
__device__ __forceinline__ uint32_t bin_start(uint32_t d, uint32_t mul)
{
    return (uint32_t)((((unsigned long long)d << 32) + mul - 1u) / mul);
}

constexpr int FINE_SHIFT = 18;                  // 32 fine bins per octave
constexpr int FINE_BINS = 256;                  // the 8 octaves of the window
__device__ __forceinline__ void bracket_from_fine(const uint32_t *fh, uint32_t n_over, FastLine &f, int t, int m, int lane)
{
    uint32_t c[8], mine = 0u;
#pragma unroll
    for (int i = 0; i < 8; ++i) { c[i] = fh[lane * 8 + i]; mine += c[i]; }
    uint32_t v = mine;                                // becomes the sum over lanes >= this one
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t u = __shfl_down_sync(FULL_MASK, v, off);
        if (lane + off < 32) v += u;
    }
    // C(b) = sample keys in fine bin b or higher; walking this lane's bins from the top
    int cum = (int)(n_over + (v - mine));
    int b_hi = FINE_BINS, b_lo = 0;                   // min{b : C(b) < t - m} (C(256) = n_over);  max{b : C(b) >= t + m}
    if (cum < t - m) b_hi = lane * 8 + 8;
#pragma unroll
    for (int i = 7; i >= 0; --i) {
        cum += (int)c[i];
        const int b = lane * 8 + i;
        if (cum < t - m) b_hi = b;
        if (cum >= t + m && b > b_lo) b_lo = b;       // first hit from the top is the largest b
    }
    b_hi = __reduce_min_sync(FULL_MASK, b_hi);
    b_lo = __reduce_max_sync(FULL_MASK, b_lo);
    if (lane == 0) {
        const uint32_t wlo = f.lo;
        f.lo = wlo + ((uint32_t)b_lo << FINE_SHIFT);
        f.hi = wlo + ((uint32_t)b_hi << FINE_SHIFT);
        f.mul = bin_multiplier(f.hi - f.lo);
        f.hi = f.lo + bin_start((uint32_t)BBINS, f.mul);   // widened to the whole histogram: "inside" is "bin below BBINS"
    }
}

// One warp: the bin of the window's histogram that holds the line's last survivor.
__device__ __forceinline__ void bracket_pick_bin(const uint32_t *h, FastLine &f, uint32_t k, int lane, int64_t L_if_below = -1)
{
    constexpr int PER_LANE = BBINS / 32;
    const uint32_t *mine_bins = h + lane * PER_LANE;
    uint32_t lane_sum = 0u;
#pragma unroll 4
    for (int i = 0; i < PER_LANE; ++i) lane_sum += mine_bins[(i + lane) & (PER_LANE - 1)];
    uint32_t v = lane_sum;                            // becomes the sum over lanes >= this one
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t t = __shfl_down_sync(FULL_MASK, v, off);
        if (lane + off < 32) v += t;
    }
    const uint32_t total = __shfl_sync(FULL_MASK, v, 0);
    // the elements above the bracket: counted directly, or what is left of the line after those below and inside it
    const uint32_t above_all = L_if_below < 0 ? f.above : (uint32_t)L_if_below - f.below - total;
    const bool in_range = k > above_all && k - above_all <= total;     // the cut lies inside the bracket
    const uint32_t krem = k - above_all;
    uint32_t above = v - lane_sum;
    const bool mine = in_range && above < krem && krem <= above + lane_sum;
    uint32_t d = 0u, g = 0u, bc = 0u;
    if (mine) {
        for (int i = PER_LANE - 1; i >= 0; --i) {
            const uint32_t c = mine_bins[i];
            if (krem <= above + c) { d = (uint32_t)(lane * PER_LANE + i); g = above; bc = c; break; }
            above += c;
        }
    }
    const uint32_t who = __ballot_sync(FULL_MASK, mine);
    const int src = who ? __ffs(who) - 1 : 0;
    const uint32_t digit = __shfl_sync(FULL_MASK, d, src);
    const uint32_t greater = __shfl_sync(FULL_MASK, g, src);
    const uint32_t bucket = __shfl_sync(FULL_MASK, bc, src);
    if (lane == 0) {
        if (!in_range || who == 0u || bucket > (uint32_t)CAND_CAP) {
            f.ok = 0u;
        } else {
            f.blo = f.lo + bin_start(digit, f.mul);
            const uint32_t end = f.lo + bin_start(digit + 1u, f.mul);
            f.bhi = end < f.hi ? end : f.hi;
            f.krem2 = krem - greater;
            f.bucket = bucket;
        }
    }
}

__device__ __forceinline__ bool cand_beats(const CandSet &c, int j, int i)
{
    if (c.key[j] != c.key[i]) return c.key[j] > c.key[i];
    if (c.k64[j] != c.k64[i]) return c.k64[j] > c.k64[i];
    return c.idx[j] < c.idx[i];
}

// One warp: ranks the collected elements of the cut's bin by the full key (rounded product, exact product, lower
// index first) and states the line's rule.  The elements that share the cut's rounded product all sit in this bin,
// so whether the exact product or the index has to split them is decided here.
__device__ __forceinline__ void bracket_rank(const CandSet &c, FastLine &f, int lane)
{
    const int n = (int)f.ncoll;
    if (n != (int)f.bucket || n > CAND_CAP) { if (lane == 0) f.ok = 0u; return; }     // should not happen; be safe
    const uint32_t want = f.krem2 - 1u;               // 0-based rank of the last survivor
    int star = -1;
    uint32_t rank[(CAND_CAP + 31) / 32];
#pragma unroll
    for (int t = 0; t < (CAND_CAP + 31) / 32; ++t) {
        const int i = t * 32 + lane;
        uint32_t r = 0u;
        if (i < n)
            for (int j = 0; j < n; ++j) r += cand_beats(c, j, i) ? 1u : 0u;
        rank[t] = r;
        if (i < n && r == want) star = i;
    }
    const uint32_t who = __ballot_sync(FULL_MASK, star >= 0);
    const int src = __ffs(who) - 1;                   // exactly one element has that rank (keys are distinct)
    star = __shfl_sync(FULL_MASK, star, src < 0 ? 0 : src);
    if (who == 0u) { if (lane == 0) f.ok = 0u; return; }
    const uint32_t key_s = c.key[star], idx_s = c.idx[star];
    const unsigned long long k64_s = c.k64[star];
    bool split_p = false, split_e = false;            // some element equal in p (and in the exact product) is pruned
#pragma unroll
    for (int t = 0; t < (CAND_CAP + 31) / 32; ++t) {
        const int i = t * 32 + lane;
        if (i < n && rank[t] > want && c.key[i] == key_s) {
            split_p = true;
            if (c.k64[i] == k64_s) split_e = true;
        }
    }
    const bool any_p = __any_sync(FULL_MASK, split_p), any_e = __any_sync(FULL_MASK, split_e);
    if (lane == 0) {
        f.res.tau32 = key_s;
        f.res.exact = any_p ? 1u : 0u;
        f.res.tau64 = k64_s;
        f.res.cut = any_e ? (long long)idx_s : 0x7fffffffffffffffll;
    }
}

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
constexpr int RS_SAMPLE = 1024;                 // evenly spaced elements of a row that place its bracket
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

// ---------------------------------------------------------------- lines that are matrix columns
// One CTA per strip of 8 adjacent columns (16 bytes of every row for bf16, 32 for f32).  The strip is not cached: the
// sweep of the sampled bracket reads it once (bf16: through bulk tensor copies), and every pass of the radix select,
// where a column needs it, reads it again with one vector load per row and thread (mostly from L2).  The kernel
// publishes a LineResult per column: the bin that holds the cut (bf16), or the exact rule (tau32, exact, tau64, cut).
constexpr int COL_THREADS = 512;                // two CTAs per SM: one sweeps while the other samples, picks its bins or waits
constexpr int COL_SAMPLE = 1024;                // evenly spaced rows of a strip that place its columns' brackets
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
#pragma unroll
        for (int h = 0; h < PN_ROWS / 4; ++h) {
            const int64_t rh = r0 + 4 * h;
            if (rh >= p.rows) break;                 // warp-uniform
            const int nrows = p.rows - rh >= 4 ? 4 : (int)(p.rows - rh);
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
            const uint32_t rows4 = nrows == 4 ? 0xffffffffu : ((1u << (8 * nrows)) - 1u);
            uint32_t keep = ~bytes_of_lanes4(Z[0], Z[1], Z[2], Z[3]) & (valid * 0x01010101u) & rows4;
            if (aside[0] | aside[1] | aside[2] | aside[3]) {     // elements of undecided bins: set aside for the ranking
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t in_bin = (aside[i] | (aside[i] >> 15)) & valid & bin_cols;   // bit j = column j
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
            const bool row_live = (lane & 3) < nrows;
            if (p.mask) {
                const uint32_t word = quad_transpose(keep, sel1, sel2);
                if (quad_live && row_live) DASS_ST(&p.mask[(rh + (lane & 3)) * p.wpr + (c0 >> 5)], word);
            }
            if (p.Wp && nvalid > 0) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (i < nrows) {
                        uint4 P;
#pragma unroll
                        for (int k = 0; k < 4; ++k) wref(P, k) = wsel(v[i], k) & ~Z[i][k];
                        store_row8(p.Wp + (rh + i) * p.ld + c0, P, nvalid);
                    }
                }
            }
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

int device_sm_count();   // dass_abi.cu
cudaError_t unit_grid_setup(UnitGrid &g, CUtensorMap *map, int64_t *grid, const void *W, int64_t rows, int64_t cols, int64_t ld,
                            bool walk_down);   // prune_nm_bf16.cu

int *stage_b_status_word();   // prune_nm_bf16.cu

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

bool tile_map_bf16(CUtensorMap *map, const void *ptr, int64_t rows, int64_t cols, int64_t ld, int box_cols, int box_rows);   // calib_tc.cu

template <bool BF16, bool ALONG, bool TMA>
static cudaError_t launch_cols_as(const SelectParams &p, cudaStream_t st)
{
    static_assert(COL_SAMPLE == RS_SAMPLE, "one sample margin serves both line directions");
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

size_t select_results_bytes(int64_t cols) { return ((size_t)cols * sizeof(LineResult) + 31) / 32 * 32; }
size_t select_scale_bytes(int64_t n) { return (size_t)((n + 7) / 8 * 8) * sizeof(float); }
// [per-column results][scale vector padded to 8][count of undecided rows, 32 bytes][their indices]
// [per column: count of elements set aside][their keys][rows][stored weights]
size_t select_workspace_bytes(int64_t rows, int64_t cols, bool norm_cols)
{
    return select_results_bytes(cols) + select_scale_bytes(norm_cols ? cols : rows) + 32 + (size_t)((rows + 7) / 8 * 8) * sizeof(uint32_t) +
           (size_t)((cols + 7) / 8 * 8) * sizeof(uint32_t) * (1 + 3 * CAND_CAP);
}

cudaError_t select_unstructured_launch(const void *W, int64_t rows, int64_t cols, int64_t ld, bool bf16,
                                       const float *norm, bool norm_cols, float alpha, uint32_t k, bool line_is_row,
                                       uint32_t *mask_bits, void *W_pruned, void *workspace, cudaStream_t st)
{
    LineResult *results = static_cast<LineResult *>(workspace);
    float *scale_ws = reinterpret_cast<float *>(static_cast<unsigned char *>(workspace) + select_results_bytes(cols));
    const int64_t n_norm = norm_cols ? cols : rows;
    uint32_t *line_count = reinterpret_cast<uint32_t *>(reinterpret_cast<unsigned char *>(scale_ws) + select_scale_bytes(n_norm));
    uint32_t *line_list = line_count + 8;
    const size_t cols8 = (size_t)((cols + 7) / 8 * 8);
    CandLists cand;
    cand.count = line_list + (rows + 7) / 8 * 8;
    cand.key = cand.count + cols8;
    cand.idx = cand.key + cols8 * CAND_CAP;
    cand.raw = cand.idx + cols8 * CAND_CAP;
    const int64_t n_pad = (n_norm + 7) / 8 * 8;
    scale_vector_kernel<<<(unsigned)((n_pad + 255) / 256), 256, 0, st>>>(norm, n_norm, n_pad, (int)scale_mode_for(alpha), alpha, scale_ws);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    SelectParams p;
    p.W = W; p.Wp = W_pruned; p.mask = mask_bits; p.scale = scale_ws; p.results = results;
    p.line_count = nullptr; p.line_list = nullptr;
    p.cand_count = (!line_is_row && bf16) ? cand.count : nullptr;
    p.status = stage_b_status_word();
    p.rows = rows; p.cols = cols; p.ld = ld;
    p.wpr = (cols + 31) / 32;
    p.L = line_is_row ? cols : rows;
    p.lpad = (p.L + 7) / 8 * 8;
    p.k = k;
    p.idx_bits = 1;
    while (((int64_t)1 << p.idx_bits) < p.L) ++p.idx_bits;
    p.scale_along_line = (line_is_row == norm_cols) ? 1 : 0;   // the norm index runs along the line
    {   // four standard deviations of the rank of a sample quantile, in sample positions, plus slack
        const double q = (double)(p.L - (int64_t)k) / (double)p.L;
        p.margin = (int)std::ceil(4.0 * std::sqrt((double)RS_SAMPLE * q * (1.0 - q))) + 2;
    }
    if (line_is_row) {
        if (mask_bits) {   // the kernel writes whole bytes of real columns; the padding of each mask row must read 0
            e = cudaMemsetAsync(mask_bits, 0, (size_t)rows * p.wpr * sizeof(uint32_t), st);
            if (e != cudaSuccess) return e;
        }
        return bf16 ? launch_rows<true>(p, line_count, line_list, st) : launch_rows<false>(p, line_count, line_list, st);
    }
    e = bf16 ? launch_cols<true>(p, st) : launch_cols<false>(p, st);
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
    if (bf16)   // the TMA-fed streaming pass
        return launch_emit_stream(W, W_pruned, mask_bits, scale_ws, results, cand, rows, cols, ld, norm_cols ? 0 : 1, st);
    select_emit_cols_kernel<false><<<grid, 256, 0, st>>>(q);
    return cudaGetLastError();
}

}  // namespace dass

using namespace dass;

extern "C" dass_status dass_select_workspace_bytes(int64_t rows, int64_t cols, dass_axis norm_axis, size_t *bytes)
{
    if (!bytes) return DASS_ERR_NULL;
    if (norm_axis != DASS_AXIS_ROWS && norm_axis != DASS_AXIS_COLS) return DASS_ERR_DTYPE;
    if (rows < 1 || cols < 1) return DASS_ERR_SHAPE;
    *bytes = select_workspace_bytes(rows, cols, norm_axis == DASS_AXIS_COLS);
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
    const bool line_is_row = compare_axis == DASS_AXIS_COLS;         // the index that varies inside a line
    const int64_t L = line_is_row ? cols : rows;
    if (L >= (int64_t)1 << 31) return DASS_ERR_UNSUPPORTED;
    if (line_is_row && select_row_smem_bytes(L, bf16) > (size_t)220 * 1024) return DASS_ERR_UNSUPPORTED;   // a row line is cached in shared memory
    size_t need = 0;
    const dass_status qs = dass_select_workspace_bytes(rows, cols, norm_axis, &need);
    if (qs != DASS_OK) return qs;
    if (!workspace || workspace_bytes < need) return DASS_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 15u) return DASS_ERR_ALIGN;
    const int64_t n_prune = (int64_t)std::floor(sparsity * (double)L);
    const uint32_t k = (uint32_t)(L - n_prune);
    DASS_BOUNDS_SCOPE(bs);
    DASS_BOUNDS_ADD(bs, W, (size_t)rows * ld * (bf16 ? 2 : 4));
    DASS_BOUNDS_ADD(bs, W_pruned, (size_t)rows * ld * (bf16 ? 2 : 4));
    DASS_BOUNDS_ADD(bs, norm, (size_t)(norm_axis == DASS_AXIS_ROWS ? rows : cols) * sizeof(float));
    DASS_BOUNDS_ADD(bs, mask_bits, (size_t)rows * ((cols + 31) / 32) * sizeof(uint32_t));
    DASS_BOUNDS_ADD(bs, workspace, workspace_bytes);
    DASS_BOUNDS_COMMIT(bs, static_cast<cudaStream_t>(cuda_stream));
    if (select_unstructured_launch(W, rows, cols, ld, bf16, norm, norm_axis == DASS_AXIS_COLS, alpha, k, line_is_row,
                                   mask_bits, W_pruned, workspace,
                                   static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return DASS_ERR_CUDA;
    return DASS_OK;
}
