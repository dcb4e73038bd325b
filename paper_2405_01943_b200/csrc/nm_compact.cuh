// Compaction of the survivors of N:M groups held in registers (generic formulation: select chains, any n:m, both
// element types).  Shared by the compression kernels and by the one-pass prune kernels for the cases that have no
// tuned kernel.  Internal header.
#pragma once

#include "dass_device.cuh"

namespace dass {

// Raw bits of element j of a chunk, j only known at run time (select chain, no local memory).
template <bool BF16>
__device__ __forceinline__ uint32_t chunk_bits_dyn(const Chunk<BF16> &c, int j)
{
    if constexpr (BF16) {
        const uint32_t a = (j & 2) ? c.w[1] : c.w[0];
        const uint32_t b = (j & 2) ? c.w[3] : c.w[2];
        const uint32_t w = (j & 4) ? b : a;
        return (j & 1) ? (w >> 16) : (w & 0xffffu);
    } else {
        const uint32_t a = (j & 1) ? c.w[1] : c.w[0];
        const uint32_t b = (j & 1) ? c.w[3] : c.w[2];
        const uint32_t d = (j & 1) ? c.w[5] : c.w[4];
        const uint32_t e = (j & 1) ? c.w[7] : c.w[6];
        const uint32_t ab = (j & 2) ? b : a;
        const uint32_t de = (j & 2) ? e : d;
        return (j & 4) ? de : ab;
    }
}

template <bool BF16>
__device__ __forceinline__ void chunk_set(Chunk<BF16> &c, int j /* compile-time after unrolling */, uint32_t bits)
{
    if constexpr (BF16) {
        if (j & 1) c.w[j >> 1] = (c.w[j >> 1] & 0x0000ffffu) | (bits << 16);
        else c.w[j >> 1] = (c.w[j >> 1] & 0xffff0000u) | (bits & 0xffffu);
    } else {
        c.w[j] = bits;
    }
}

// Stores the first n elements of a chunk at element offset `off`; vector stores only if the
// destination is known to be 16-byte aligned (vec) and the piece is a whole vector.
template <bool BF16>
__device__ __forceinline__ void chunk_store_n(const Chunk<BF16> &c, void *base, int64_t off, int n, bool vec)
{
    if constexpr (BF16) {
        uint16_t *p = static_cast<uint16_t *>(base) + off;
        if (vec && n == 8) {
            DASS_ST_CS(reinterpret_cast<uint4 *>(p), make_uint4(c.w[0], c.w[1], c.w[2], c.w[3]));
        } else if (vec && n == 4) {
            DASS_ST_CS(reinterpret_cast<uint2 *>(p), make_uint2(c.w[0], c.w[1]));
        } else {
            for (int j = 0; j < n; ++j) DASS_ST(&p[j], (uint16_t)chunk_bits_dyn<true>(c, j));
        }
    } else {
        uint32_t *p = static_cast<uint32_t *>(base) + off;
        if (vec && n == 8) {
            DASS_ST_CS(reinterpret_cast<uint4 *>(p), make_uint4(c.w[0], c.w[1], c.w[2], c.w[3]));
            DASS_ST_CS(reinterpret_cast<uint4 *>(p) + 1, make_uint4(c.w[4], c.w[5], c.w[6], c.w[7]));
        } else if (vec && n == 4) {
            DASS_ST_CS(reinterpret_cast<uint4 *>(p), make_uint4(c.w[0], c.w[1], c.w[2], c.w[3]));
        } else {
            for (int j = 0; j < n; ++j) DASS_ST(&p[j], chunk_bits_dyn<false>(c, j));
        }
    }
}

// Position (0-based) of the k-th (0-based) set bit of x; x has more than k bits set.
__device__ __forceinline__ int nth_set_bit(uint32_t x, int k)
{
    for (int i = 0; i < k; ++i) x &= x - 1;
    return __ffs(x) - 1;
}

// Column groups: the 8 elements of one row (8 / M groups) and their keep byte -> the survivors in index order
// (the first nout elements of `out`) and the metadata byte (2:4: two nibbles pos_lo | pos_hi << 2, else the keep
// byte itself).
template <bool BF16, int M, bool TWO_FOUR>
__device__ __forceinline__ uint32_t compact_cols(const Chunk<BF16> &ch, uint32_t mbyte, int n_keep, int nout, Chunk<BF16> &out)
{
    chunk_zero<BF16>(out);
    if constexpr (TWO_FOUR) {
        uint32_t field_byte = 0u;
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            const uint32_t nib = (mbyte >> (4 * g)) & 0xfu;
            const int lo = nib ? __ffs(nib) - 1 : 0;
            const int hi = nib ? 31 - __clz(nib) : 0;
            chunk_set<BF16>(out, 2 * g, chunk_bits_dyn<BF16>(ch, 4 * g + lo));
            chunk_set<BF16>(out, 2 * g + 1, chunk_bits_dyn<BF16>(ch, 4 * g + hi));
            field_byte |= (uint32_t)(lo | (hi << 2)) << (4 * g);
        }
        return field_byte;
    } else {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            if (k < nout) {
                const int g = k / n_keep, q = k % n_keep;
                const uint32_t gm = (mbyte >> (g * M)) & ((1u << M) - 1u);
                chunk_set<BF16>(out, k, chunk_bits_dyn<BF16>(ch, g * M + nth_set_bit(gm, q)));
            }
        }
        return mbyte;   // the m-bit keep masks, already in place
    }
}

// Row groups: M rows at a lane's 8 columns and their keep bytes -> up to MAXK output rows (survivor k of every
// column) and the packed fields of the 8 columns (4-bit fields: all in fields_lo; 8-bit fields: columns 0..3 in
// fields_lo, 4..7 in fields_hi).
template <bool BF16, int M, bool TWO_FOUR, int MAXK>
__device__ __forceinline__ void compact_rows(const Chunk<BF16> (&ch)[M], const uint32_t (&mbyte)[M], int n_keep,
                                             Chunk<BF16> (&out)[MAXK], uint32_t &fields_lo, uint32_t &fields_hi)
{
#pragma unroll
    for (int k = 0; k < MAXK; ++k) chunk_zero<BF16>(out[k]);
    fields_lo = 0u;
    fields_hi = 0u;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        uint32_t colmask = 0u;   // bit q: row q kept at column j
#pragma unroll
        for (int q = 0; q < M; ++q) colmask |= ((mbyte[q] >> j) & 1u) << q;
        if constexpr (TWO_FOUR) {
            const int lo = colmask ? __ffs(colmask) - 1 : 0;
            const int hi = colmask ? 31 - __clz(colmask) : 0;
            const uint32_t v_lo = lo == 0 ? chunk_bits<BF16>(ch[0], j) : lo == 1 ? chunk_bits<BF16>(ch[1], j)
                                : lo == 2 ? chunk_bits<BF16>(ch[2], j) : chunk_bits<BF16>(ch[3], j);
            const uint32_t v_hi = hi == 0 ? chunk_bits<BF16>(ch[0], j) : hi == 1 ? chunk_bits<BF16>(ch[1], j)
                                : hi == 2 ? chunk_bits<BF16>(ch[2], j) : chunk_bits<BF16>(ch[3], j);
            chunk_set<BF16>(out[0], j, v_lo);
            chunk_set<BF16>(out[1], j, v_hi);
            fields_lo |= (uint32_t)(lo | (hi << 2)) << (4 * j);
        } else {
#pragma unroll
            for (int k = 0; k < MAXK; ++k) {
                if (k < n_keep) {
                    const int pos = nth_set_bit(colmask, k);
                    uint32_t v = 0u;
#pragma unroll
                    for (int q = 0; q < M; ++q) v = pos == q ? chunk_bits<BF16>(ch[q], j) : v;
                    chunk_set<BF16>(out[k], j, v);
                }
            }
            if constexpr (M == 4) fields_lo |= colmask << (4 * j);
            else if (j < 4) fields_lo |= colmask << (8 * j);
            else fields_hi |= colmask << (8 * (j - 4));
        }
    }
}

}  // namespace dass
