// Shared device-side helpers of the DaSS CUDA library (element access, the norm^alpha recipe,
// exact score keys).  Internal header; the public boundary is include/dass.h.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "dass.h"
#include "bounds_check.cuh"

namespace dass {

constexpr unsigned FULL_MASK = 0xffffffffu;

// How ||y||^alpha of Eq. 4 is evaluated (chosen on the host from alpha).  The listed exponents use
// only correctly rounded IEEE operations in double followed by one rounding to float, so the value
// is reproducible bit for bit on any IEEE machine.
enum ScaleMode : int {
    SCALE_ONE = 0,      // alpha == 0      -> 1 (also for a zero norm: 0^0 := 1)
    SCALE_IDENTITY = 1, // alpha == 1      -> n
    SCALE_SQRT = 2,     // alpha == 1/2    -> sqrt(n)
    SCALE_QRT = 3,      // alpha == 1/4    -> sqrt(sqrt(n))
    SCALE_3QRT = 4,     // alpha == 3/4    -> sqrt(n) * sqrt(sqrt(n))
    SCALE_POW = 5       // anything else   -> pow(n, alpha)
};

inline ScaleMode scale_mode_for(float alpha)
{
    if (alpha == 0.0f) return SCALE_ONE;
    if (alpha == 1.0f) return SCALE_IDENTITY;
    if (alpha == 0.5f) return SCALE_SQRT;
    if (alpha == 0.25f) return SCALE_QRT;
    if (alpha == 0.75f) return SCALE_3QRT;
    return SCALE_POW;
}

__device__ __forceinline__ float scale_from_norm(float n, int mode, float alpha)
{
    const double x = (double)n;
    switch (mode) {
    case SCALE_ONE: return 1.0f;
    case SCALE_IDENTITY: return n;
    case SCALE_SQRT: return __double2float_rn(sqrt(x));
    case SCALE_QRT: return __double2float_rn(sqrt(sqrt(x)));
    case SCALE_3QRT: {
        const double r = sqrt(x);
        const double q = sqrt(r);
        return __double2float_rn(__dmul_rn(r, q));
    }
    default: return __double2float_rn(pow(x, (double)alpha));
    }
}

// A chunk of 8 consecutive elements of one matrix row, kept as raw bits.
// bf16: 4 words (two elements per word, lower column in the low half); f32: 8 words.
template <bool BF16>
struct Chunk {
    static constexpr int WORDS = BF16 ? 4 : 8;
    uint32_t w[WORDS];
};

template <bool BF16>
__device__ __forceinline__ void chunk_zero(Chunk<BF16> &c)
{
#pragma unroll
    for (int i = 0; i < Chunk<BF16>::WORDS; ++i) c.w[i] = 0u;
}

// Loads the chunk that starts at element `off` of `base` (off is a multiple of 8 elements and the
// row pitch is a multiple of 16 bytes, so every 16-byte load is aligned).  `nvalid` (1..8) elements
// exist; a bf16 row is padded to 8 elements by its pitch so one vector load stays inside the row,
// an f32 row only to 4, so the second vector is read only when it holds a valid element.
template <bool BF16>
__device__ __forceinline__ void chunk_load(Chunk<BF16> &c, const void *base, int64_t off, int nvalid)
{
    if constexpr (BF16) {
        const uint4 v = DASS_LD_CS(reinterpret_cast<const uint4 *>(static_cast<const uint16_t *>(base) + off));
        c.w[0] = v.x; c.w[1] = v.y; c.w[2] = v.z; c.w[3] = v.w;
    } else {
        const uint4 *p = reinterpret_cast<const uint4 *>(static_cast<const uint32_t *>(base) + off);
        const uint4 a = DASS_LD_CS(p);
        c.w[0] = a.x; c.w[1] = a.y; c.w[2] = a.z; c.w[3] = a.w;
        if (nvalid > 4) {
            const uint4 b = DASS_LD_CS(p + 1);
            c.w[4] = b.x; c.w[5] = b.y; c.w[6] = b.z; c.w[7] = b.w;
        } else {
            c.w[4] = c.w[5] = c.w[6] = c.w[7] = 0u;
        }
    }
}

// |element j| widened to float (exact for both types).
template <bool BF16>
__device__ __forceinline__ float chunk_abs(const Chunk<BF16> &c, int j)
{
    if constexpr (BF16) {
        const uint32_t word = c.w[j >> 1];
        const uint32_t bits = (j & 1) ? (word & 0x7fff0000u) : ((word & 0x00007fffu) << 16);
        return __uint_as_float(bits);
    } else {
        return __uint_as_float(c.w[j] & 0x7fffffffu);
    }
}

// Raw bits of element j (16 bits for bf16, 32 for f32).
template <bool BF16>
__device__ __forceinline__ uint32_t chunk_bits(const Chunk<BF16> &c, int j)
{
    if constexpr (BF16) return (j & 1) ? (c.w[j >> 1] >> 16) : (c.w[j >> 1] & 0xffffu);
    else return c.w[j];
}

// Zeroes (+0) every element whose bit in `keep` (bit j = element j) is clear.
template <bool BF16>
__device__ __forceinline__ void chunk_apply_mask(Chunk<BF16> &c, uint32_t keep)
{
    if constexpr (BF16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t lo = (keep >> (2 * i)) & 1u ? 0x0000ffffu : 0u;
            const uint32_t hi = (keep >> (2 * i + 1)) & 1u ? 0xffff0000u : 0u;
            c.w[i] &= (lo | hi);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) c.w[i] = (keep >> i) & 1u ? c.w[i] : 0u;
    }
}

// Stores the first `nvalid` elements of the chunk at element `off` of `base`.
template <bool BF16>
__device__ __forceinline__ void chunk_store(const Chunk<BF16> &c, void *base, int64_t off, int nvalid)
{
    if constexpr (BF16) {
        uint16_t *p = static_cast<uint16_t *>(base) + off;
        if (nvalid == 8) {
            DASS_ST_CS(reinterpret_cast<uint4 *>(p), make_uint4(c.w[0], c.w[1], c.w[2], c.w[3]));
        } else {
            for (int j = 0; j < nvalid; ++j) DASS_ST(&p[j], (uint16_t)chunk_bits<true>(c, j));
        }
    } else {
        uint32_t *p = static_cast<uint32_t *>(base) + off;
        if (nvalid >= 4) DASS_ST_CS(reinterpret_cast<uint4 *>(p), make_uint4(c.w[0], c.w[1], c.w[2], c.w[3]));
        if (nvalid == 8) {
            DASS_ST_CS(reinterpret_cast<uint4 *>(p) + 1, make_uint4(c.w[4], c.w[5], c.w[6], c.w[7]));
        } else {
            for (int j = (nvalid >= 4 ? 4 : 0); j < nvalid; ++j) DASS_ST(&p[j], c.w[j]);
        }
    }
}

// Combines the byte each lane of a quad (4 consecutive lanes) holds into the 32-bit word covering
// the quad's 32 columns; valid in every lane afterwards.  Must be called by the whole warp.
__device__ __forceinline__ uint32_t quad_pack_bytes(uint32_t byte, int lane)
{
    uint32_t v = byte << (8 * (lane & 3));
    v |= __shfl_xor_sync(FULL_MASK, v, 1);
    v |= __shfl_xor_sync(FULL_MASK, v, 2);
    return v;
}

// Keep flags of one group of M scores: element p is kept iff fewer than n_keep elements precede it
// in the order "higher score first, lower index first".  One comparison per pair.
template <int M>
__device__ __forceinline__ uint32_t select_group(const double (&s)[M], int n_keep)
{
    int rank[M];
#pragma unroll
    for (int p = 0; p < M; ++p) rank[p] = 0;
#pragma unroll
    for (int a = 0; a < M; ++a) {
#pragma unroll
        for (int b = a + 1; b < M; ++b) {
            const bool b_first = s[b] > s[a];   // ties: the lower index a stays ahead
            rank[a] += b_first ? 1 : 0;
            rank[b] += b_first ? 0 : 1;
        }
    }
    uint32_t keep = 0;
#pragma unroll
    for (int p = 0; p < M; ++p) keep |= (rank[p] < n_keep ? 1u : 0u) << p;
    return keep;
}

}  // namespace dass
