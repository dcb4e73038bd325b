// Shared by the sources of the unstructured selection (select_unstructured.cu, select_rows.cu, select_cols.cu,
// select_emit.cu): what a decided line looks like, the parameters of the kernels, the radix select on the three-part
// key, and the sampled bracket (window, fine histogram, bin of the cut, ranking of the bin's elements).  Internal header.
#pragma once

#include <cmath>
#include <cstring>
#include <type_traits>

#include "stream_units.cuh"

namespace dass {

constexpr int SELECT_SAMPLE = 1024;             // evenly spaced elements of a line that place its bracket (both line directions)

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
    int margin;             // sampled bracket: sample positions on either side of the wanted rank (five standard deviations)
    uint32_t *line_count;   // row lines: how many lines the streaming kernel left undecided, and which
    uint32_t *line_list;    // (both null: the radix kernel takes every row)
    uint32_t *cand_count;   // column lines, bf16: per-column count of the elements the emit pass sets aside (cleared here)
    int *status;            // device status word for bounded waits that ran out
};


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
// off the expected rank (m is five standard deviations of that rank, set by the host); the bracket is those two
// keys' fine bins and what lies between.  About 2m/S of the line plus two fine bins falls inside; everything else
// is only counted.  A miss shows in bracket_pick_bin's counts and sends the line to the radix select.
// Bins of the bracket's histogram: BBINS of them (about a fifth of a line falls inside the bracket: 5 elements per bin
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

// ---------------------------------------------------------------- host side, one launcher per source file
int device_sm_count();                            // dass_abi.cu
int *stage_b_status_word();                       // prune_nm_bf16.cu
cudaError_t unit_grid_setup(UnitGrid &g, CUtensorMap *map, int64_t *grid, const void *W, int64_t rows, int64_t cols, int64_t ld,
                            bool walk_down);      // prune_nm_bf16.cu
bool tile_map_bf16(CUtensorMap *map, const void *ptr, int64_t rows, int64_t cols, int64_t ld, int box_cols, int box_rows);   // calib_tc.cu

size_t select_row_smem_bytes(int64_t L, bool bf16);                                                   // select_rows.cu
cudaError_t select_launch_rows(const SelectParams &p, bool bf16, uint32_t *line_count, uint32_t *line_list, cudaStream_t st);   // select_rows.cu
cudaError_t select_launch_cols(const SelectParams &p, bool bf16, cudaStream_t st);                    // select_cols.cu
cudaError_t select_launch_emit(const SelectParams &p, bool bf16, const CandLists &cand, int scale_per_row, cudaStream_t st);    // select_emit.cu

}  // namespace dass
