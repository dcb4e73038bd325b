// Building blocks of the streaming stage-(b) kernels that are fed by TMA (the one-pass N:M kernels, the emit pass of
// the unstructured selection): the decomposition of a matrix into warp units of 8 rows x 256 columns and runs of
// units, the per-warp ring of TMA boxes, and the lane-mask / byte helpers of a lane's 8 x 8 tile.  Internal header.
#pragma once

#include "tc_common.cuh"

namespace dass {

// How a matrix is cut into units and runs (filled by unit_grid_setup on the host).
struct UnitGrid {
    int64_t rows, cols;
    int64_t strips, blocks;          // 256-column strips, 8-row blocks
    int64_t fast;        // units along the direction a warp walks (the scales stay the same along it)
    int runs;            // a line of `fast` units is cut into this many near-equal runs, one per warp
    int ctas_per_line;   // per-column scales: CTAs that share one strip (runs / warps per CTA, rounded up)
    uint32_t box_bytes;  // bytes of one TMA box (box columns x box rows x 2)
    uint32_t pitch16;    // row pitch of a box in shared memory, in 16-byte vectors
    int *status;         // device word that receives DASS_ERR_TIMEOUT when a bounded wait runs out
};

constexpr int PN_THREADS = 128;
constexpr int PN_MIN_BLOCKS = 4;     // 16 warps per SM at up to 128 registers
constexpr int PN_COLS = 256;
constexpr int PN_ROWS = 8;

// Out of line: the double-precision sqrt / pow sequences run once per strip or per 32 rows only.
static __device__ __noinline__ float pn_scale_of(float n, int mode, float alpha) { return scale_from_norm(n, mode, alpha); }

__device__ __forceinline__ uint32_t pn_prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

__device__ __forceinline__ float max3f(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

__device__ __forceinline__ uint32_t wsel(const uint4 &v, int k) { return k == 0 ? v.x : k == 1 ? v.y : k == 2 ? v.z : v.w; }
__device__ __forceinline__ uint32_t &wref(uint4 &v, int k) { return k == 0 ? v.x : k == 1 ? v.y : k == 2 ? v.z : v.w; }

// fl32(|low bf16 of word| * s) and the same for the high one.  The low half is moved up with a multiply so that it
// runs beside the float pipe rather than on the logic pipe.
__device__ __forceinline__ float prod_lo(uint32_t word, float s) { return fabsf(__uint_as_float(word * 65536u)) * s; }
__device__ __forceinline__ float prod_hi(uint32_t word, float s) { return fabsf(__uint_as_float(word & 0xffff0000u)) * s; }

// Second largest of four.
__device__ __forceinline__ float cut_2of4(float a, float b, float c, float d)
{
    const float h1 = fmaxf(a, b), l1 = fminf(a, b), h2 = fmaxf(c, d), l2 = fminf(c, d);
    return max3f(fminf(h1, h2), l1, l2);
}

__device__ __forceinline__ void sort4_desc(float &a, float &b, float &c, float &d)
{
    const float h1 = fmaxf(a, b), l1 = fminf(a, b), h2 = fmaxf(c, d), l2 = fminf(c, d);
    const float m = fminf(h1, h2), l = fmaxf(l1, l2);
    a = fmaxf(h1, h2);
    b = fmaxf(m, l);
    c = fminf(m, l);
    d = fminf(l1, l2);
}

// Fourth largest of eight: both halves sorted, then the merge rule "the k-th largest of two sorted lists is the
// largest of min(a_i, b_(k-2-i)) and of a_(k-1), b_(k-1)".
__device__ __forceinline__ float cut_4of8(const float (&x)[8])
{
    float a0 = x[0], a1 = x[1], a2 = x[2], a3 = x[3], b0 = x[4], b1 = x[5], b2 = x[6], b3 = x[7];
    sort4_desc(a0, a1, a2, a3);
    sort4_desc(b0, b1, b2, b3);
    return max3f(max3f(a3, b3, fminf(a0, b2)), fminf(a1, b1), fminf(a2, b0));
}

template <int M>
__device__ __forceinline__ float cut_of(const float (&x)[M])
{
    if constexpr (M == 4) return cut_2of4(x[0], x[1], x[2], x[3]);
    else return cut_4of8(x);
}

// Lane mask of a word from the differences of its two elements: 0xffff where the difference is negative.
__device__ __forceinline__ uint32_t pruned_lanes(float d_lo, float d_hi)
{
    return pn_prmt(__float_as_uint(d_lo), __float_as_uint(d_hi), 0xFFBBu);
}

// Bytes (bit j = column j) of the lane-mask words of two rows, in the low 16 bits of the result (row a in byte 0,
// row b in byte 1).  Even columns sit in the low lanes and land on their bit directly; odd columns sit in the high
// lanes, are picked 16 bits up and folded down at the end.
__device__ __forceinline__ uint32_t bytes_of_lanes2(const uint32_t (&za)[4], const uint32_t (&zb)[4])
{
    uint32_t x = za[0] & 0x00020001u;
    x |= za[1] & 0x00080004u;
    x |= za[2] & 0x00200010u;
    x |= za[3] & 0x00800040u;
    x |= zb[0] & 0x02000100u;
    x |= zb[1] & 0x08000400u;
    x |= zb[2] & 0x20001000u;
    x |= zb[3] & 0x80004000u;
    return x | (x >> 16);
}

// "Pruned" bytes of four rows in one word (byte i = row i).
__device__ __forceinline__ uint32_t bytes_of_lanes4(const uint32_t (&z0)[4], const uint32_t (&z1)[4], const uint32_t (&z2)[4],
                                                    const uint32_t (&z3)[4])
{
    return pn_prmt(bytes_of_lanes2(z0, z1), bytes_of_lanes2(z2, z3), 0x5410u);
}

// 16-bit lane masks (0xffff per set bit) of an 8-bit byte: bit j -> sign of byte j, then sign-replicating permutes.
__device__ __forceinline__ void lanes_of_byte(uint32_t byte, uint32_t (&m)[4])
{
    const uint32_t zlo = (byte & 0xfu) * 0x10204080u;
    const uint32_t zhi = ((byte >> 4) & 0xfu) * 0x10204080u;
    m[0] = pn_prmt(zlo, 0u, 0x9988u);
    m[1] = pn_prmt(zlo, 0u, 0xbbaau);
    m[2] = pn_prmt(zhi, 0u, 0x9988u);
    m[3] = pn_prmt(zhi, 0u, 0xbbaau);
}

// 4 x 4 byte transpose across a quad of lanes: on entry byte i of x belongs to row i (this lane's 8 columns); on
// return lane k of the quad holds the word of row k (byte l from lane l of the quad).  Whole warp must call.
__device__ __forceinline__ uint32_t quad_transpose(uint32_t x, uint32_t sel1, uint32_t sel2)
{
    const uint32_t y = __shfl_xor_sync(FULL_MASK, x, 1);
    const uint32_t z = pn_prmt(x, y, sel1);
    const uint32_t y2 = __shfl_xor_sync(FULL_MASK, z, 2);
    return pn_prmt(z, y2, sel2);
}

// Stores the first n of a lane's 8 elements; one 16-byte store when all 8 exist and the address is known to be aligned.
__device__ __forceinline__ void store_row8(uint16_t *dst, const uint4 &v, int n, bool vec = true)
{
    if (vec && n == 8) {
        DASS_ST_CS(reinterpret_cast<uint4 *>(dst), v);
    } else {
        for (int j = 0; j < n; ++j) {
            const uint32_t w = wsel(v, j >> 1);
            DASS_ST(&dst[j], (uint16_t)((j & 1) ? (w >> 16) : (w & 0xffffu)));
        }
    }
}

// ---------------------------------------------------------------- work decomposition
// A unit is 8 rows x 256 columns.  A warp walks a run of consecutive units in the direction along which its
// scales stay the same: down a strip when the scales belong to columns, across the strips of one 8-row block when
// they belong to rows.  A line of units along that direction is cut into p.runs near-equal runs.  CTAs are small
// (4 warps, a few units per warp) and numerous, so the hardware's block scheduler evens out the SMs.
//   per-column scales: the warps of a CTA take consecutive runs of ONE strip and share its 256 scales through
//                      shared memory;
//   per-row scales:    the warps of a CTA take the same strip range at consecutive row blocks.
constexpr int PN_STAGES = 3;
constexpr uint32_t PN_SLOT_BYTES = PN_ROWS * PN_COLS * 2;           // 4 KB: one full box
constexpr uint32_t PN_WARPS = PN_THREADS / 32;
constexpr uint32_t pn_smem_bytes(int stages) { return PN_WARPS * stages * PN_SLOT_BYTES + PN_WARPS * stages * 8 + 128; }
constexpr uint32_t PN_SMEM_BYTES = pn_smem_bytes(PN_STAGES);
constexpr unsigned long long PN_WAIT_NS = 2000000000ull;            // a wait gives up after 2 s

template <bool NORM_COLS>
struct Run {
    int line;        // the fixed index: strip (per-column scales) or row block (per-row scales)
    int f0, f1;      // units [f0, f1) along the walking direction; empty for a warp without work
    __device__ __forceinline__ void set(const UnitGrid &p, int warp_in_cta)
    {
        int r;
        bool live;
        if constexpr (NORM_COLS) {
            line = (int)(blockIdx.x / (unsigned)p.ctas_per_line);
            r = (int)(blockIdx.x % (unsigned)p.ctas_per_line) * (int)PN_WARPS + warp_in_cta;
            live = r < p.runs;
        } else {
            line = (int)(blockIdx.x / (unsigned)p.runs) * (int)PN_WARPS + warp_in_cta;
            r = (int)(blockIdx.x % (unsigned)p.runs);
            live = line < p.blocks;
        }
        f0 = live ? (int)((int64_t)r * p.fast / p.runs) : 0;
        f1 = live ? (int)((int64_t)(r + 1) * p.fast / p.runs) : 0;
    }
    __device__ __forceinline__ int strip(int f) const { return NORM_COLS ? line : f; }
    __device__ __forceinline__ int blk(int f) const { return NORM_COLS ? f : line; }
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y) : "memory");
}

// Bounded wait of the whole warp on one of its slots.  False after PN_WAIT_NS.
__device__ __forceinline__ bool slot_wait(uint32_t bar, uint32_t parity)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t spin = 1; spin < (1u << 30); ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 63u) == 0 && global_ns() - t0 > PN_WAIT_NS) return false;
    }
    return false;
}

// The TMA-fed ring of a warp: STAGES slots of one box each, one mbarrier per slot.
template <bool NORM_COLS, int STAGES = PN_STAGES>
struct UnitRing {
    uint32_t slots, bars;            // shared-memory addresses of this warp's slots and barriers
    const uint8_t *generic;          // generic pointer to slot 0
    int f_pre;                       // next unit of the run to fetch
    int slot = 0;
    uint32_t phase = 0;

    __device__ __forceinline__ void issue(const CUtensorMap *map, const UnitGrid &p, const Run<NORM_COLS> &run, int into, int lane)
    {
        if (lane == 0 && f_pre < run.f1) {
            const uint32_t bar = bars + 8u * into;
            mbar_arrive_expect_tx(bar, p.box_bytes);
            tma_load_2d(slots + into * PN_SLOT_BYTES, map, bar, run.strip(f_pre) * PN_COLS, run.blk(f_pre) * PN_ROWS);
        }
        ++f_pre;
    }
    __device__ __forceinline__ void start(uint8_t *smem_aligned, int warp_in_cta, const CUtensorMap *map, const UnitGrid &p,
                                          const Run<NORM_COLS> &run, int lane)
    {
        generic = smem_aligned + warp_in_cta * STAGES * PN_SLOT_BYTES;
        slots = smem_u32(generic);
        bars = smem_u32(smem_aligned + PN_WARPS * STAGES * PN_SLOT_BYTES) + warp_in_cta * STAGES * 8;
        if (lane == 0) {
#pragma unroll
            for (int s = 0; s < STAGES; ++s) mbar_init(bars + 8u * s, 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
        f_pre = run.f0;
#pragma unroll
        for (int s = 0; s < STAGES - 1; ++s) issue(map, p, run, s, lane);
    }
    // Refills the slot consumed one iteration ago, then waits for the current unit.  Returns its tile (16-byte
    // vectors, row pitch p.pitch16) or nullptr when the wait ran out.
    __device__ __forceinline__ const uint4 *next(const CUtensorMap *map, const UnitGrid &p, const Run<NORM_COLS> &run, int lane)
    {
        __syncwarp();                  // every lane is done reading the slot that is refilled now
        issue(map, p, run, slot == 0 ? STAGES - 1 : slot - 1, lane);
        const bool ok = slot_wait(bars + 8u * slot, phase);
        const uint4 *tile = reinterpret_cast<const uint4 *>(generic + slot * PN_SLOT_BYTES);
        if (++slot == STAGES) { slot = 0; phase ^= 1u; }
        return ok ? tile : nullptr;
    }
    // After a failed wait: record it and give the copies still in flight one more bounded chance to land.
    __device__ __forceinline__ void fail(int lane, int *status)
    {
        if (lane == 0 && status) atomicMax(status, (int)DASS_ERR_TIMEOUT);
#pragma unroll
        for (int s = 0; s < STAGES; ++s) {
            slot_wait(bars + 8u * s, 0u);
            slot_wait(bars + 8u * s, 1u);
        }
    }
};

}  // namespace dass
