// Forward pass of the (pruned) GLU MLP layer for bf16 tensors, Eq. 2 then Eq. 3, on the sm_100a tensor cores:
//
//   kernel <MODE_GLU>    H[t, i] = bf16( act(x_t . Wg_i) * (x_t . Wu_i) )          (Eq. 2)
//   kernel <MODE_PLAIN>  Z[t, n] = bf16( h_t . Wd_n )                               (Eq. 3)
//
// Both are one persistent, warp-specialised kernel run by CTA pairs (a cluster of 2 = the two SMs of a TPC) that
// drive tcgen05.mma.cta_group::2 of shape 256 x 256 x 16:
//   * M = tokens: each CTA of the pair owns 128 tokens (TMEM lanes) and loads their 128 x 64 slice of the left
//     operand (X, or H for Eq. 3);
//   * N = 256 output columns, of which each CTA loads half of the right operand: for Eq. 2 the leader loads 128
//     rows of Wg and its peer the same 128 rows of Wu, so accumulator columns 0..127 hold the gate and 128..255
//     the up projection of the same neurons; for Eq. 3 the halves are consecutive 128-row blocks of Wd;
//   * an accumulator is 256 TMEM columns, so two fit: the epilogue of one tile (tcgen05.ld, activation and gating
//     product, rounding to bf16, 16-byte stores: a thread owns one token row, its outputs are contiguous) runs
//     while the MMAs of the next tile fill the other.
//   warp 0      TMA producer into a 6-stage, 128B-swizzled shared-memory ring (no multicast)
//   warp 1      allocates TMEM; in the leader CTA one lane issues the MMAs and commits ring slots / accumulators
//   warps 2..5  epilogue
// Work items are (output tile, band of token tiles), ordered so that the pairs running together share a few
// operand tiles through L2; the producers re-align at tile boundaries with a bounded counting barrier, right
// operand loads are evict-last and left operand loads evict-first, as in the calibration kernel.  Pruned weights
// are zeros stored in place, so the dense contraction is the pruned layer.
//
// Every wait on an mbarrier is bounded: when one runs out the CTA raises an abort flag, records
// DASS_ERR_TIMEOUT in the status word, lets its roles drain and frees its TMEM before returning.
#include "tc_common.cuh"
#include "tc_pair.cuh"

namespace dass {

constexpr int FW_BM = 128;         // tokens per CTA (256 per pair): MMA M / 2, TMEM lanes
constexpr int FW_BN = 256;         // accumulator columns per tile (MMA N); each CTA loads 128 right-operand rows
constexpr int FW_BK = 64;          // k per ring slot: 64 bf16 = one 128-byte swizzle row
constexpr int FW_UMMA_K = 16;
constexpr int FW_STAGES = 6;
constexpr int FW_ACC_STAGES = 2;   // accumulators in TMEM
constexpr unsigned long long FW_ALIGN_NS = 20000ull;
constexpr int FW_THREADS = 192;
constexpr uint32_t FW_TILE_BYTES = 128 * FW_BK * 2;                // 16 KB: a 128-row, 64-column bf16 tile
constexpr uint32_t FW_STAGE_BYTES = 2 * FW_TILE_BYTES;             // left + right = 32 KB per CTA
constexpr uint32_t FW_TMEM_COLS = FW_ACC_STAGES * FW_BN;           // 512
constexpr uint32_t FW_SMEM_BYTES = FW_STAGES * FW_STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;

constexpr int MODE_GLU = 0, MODE_PLAIN = 1;

struct FwParams {
    uint16_t *out;        // [T x n_out] bf16, pitch ldo
    int64_t ldo;
    int *status;          // device status word (0 = ok)
    int *align_counter;   // arrivals of the tile-boundary alignment barrier (zero before the launch)
    int64_t T;            // tokens
    int64_t n_out;        // output columns: I (MODE_GLU) or d (MODE_PLAIN)
    int64_t out_tile;     // output columns per item: 128 (MODE_GLU) or 256 (MODE_PLAIN)
    int64_t peer_row_offset;   // right-operand row offset of the peer's half inside its tensor map: 0 or 128
    int64_t out_tiles, token_tiles, bands, items, k_blocks;
    int band_tiles;       // token tiles per band
    int super_bands;      // bands interleaved in the item order
    int vector_ok;        // out is 16-byte aligned and ldo a multiple of 8: whole 16-byte stores
};

struct FwItem { int64_t ot, band; };

__device__ __forceinline__ FwItem fw_decode_item(const FwParams &p, int64_t idx)
{
    const int64_t per_super = p.out_tiles * p.super_bands;
    const int64_t sb = idx / per_super;
    const int64_t rem = idx - sb * per_super;
    const int64_t left = p.bands - sb * p.super_bands;
    const int64_t nb = left < p.super_bands ? left : p.super_bands;
    FwItem c;
    c.ot = rem / nb;
    c.band = sb * p.super_bands + (rem - c.ot * nb);
    return c;
}

__device__ __forceinline__ uint32_t fw_pack_bf16(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));     // first source -> upper half
    return r;
}

// Stores 32 consecutive outputs of one token row (packed two per word, lower column in the low half) starting
// at column n0; columns at and past n_out do not exist.
__device__ __forceinline__ void fw_store_32(const FwParams &p, uint16_t *row, int64_t n0, const uint32_t (&w)[16])
{
    if (p.vector_ok && n0 + 32 <= p.n_out) {
        uint4 *dst = reinterpret_cast<uint4 *>(row + n0);               // n0 is a multiple of 32
#pragma unroll
        for (int v = 0; v < 4; ++v) DASS_ST(&dst[v], make_uint4(w[4 * v], w[4 * v + 1], w[4 * v + 2], w[4 * v + 3]));
    } else {
#pragma unroll
        for (int j = 0; j < 32; ++j)
            if (n0 + j < p.n_out) DASS_ST(&row[n0 + j], (uint16_t)((j & 1) ? (w[j >> 1] >> 16) : (w[j >> 1] & 0xffffu)));
    }
}

template <int MODE, int ACT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(FW_THREADS, 1)
mlp_forward_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b0,
                      const __grid_constant__ CUtensorMap map_b1, const FwParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;                 // swizzled tiles need 1024-byte alignment
    uint8_t *aligned = smem_raw + (base - raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(aligned + FW_STAGES * FW_STAGE_BYTES);
    const uint32_t bar_full = smem_u32(bars);                     // [FW_STAGES], used in the leader CTA only
    const uint32_t bar_empty = bar_full + 8 * FW_STAGES;          // [FW_STAGES], one set per CTA
    const uint32_t bar_acc_full = bar_empty + 8 * FW_STAGES;      // [FW_ACC_STAGES], per CTA
    const uint32_t bar_acc_empty = bar_acc_full + 8 * FW_ACC_STAGES;   // [FW_ACC_STAGES], leader only: 8 epilogue warps arrive
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * FW_STAGES + 2 * FW_ACC_STAGES);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                      // 0 = leader
    const int64_t cluster_id = blockIdx.x >> 1;
    const int64_t nclusters = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < FW_STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int s = 0; s < FW_ACC_STAGES; ++s) {
            mbar_init(bar_acc_full + 8 * s, 1);
            mbar_init(bar_acc_empty + 8 * s, 8);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(tmem_slot), FW_TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();            // both CTAs' barriers are initialised and both TMEM allocations exist
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (one per CTA)
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            // a right-operand tile is re-read for every token tile of a band: keep it in L2; a left-operand tile
            // is shared only by the pairs reading it right now: let it go first
            const uint64_t pol_b = l2_policy_evict_last();
            const uint64_t pol_a = l2_policy_evict_first();
            const uint32_t leader_full = map_to_cta(bar_full, 0);
            const CUtensorMap *map_b = rank ? &map_b1 : &map_b0;
            int64_t round = 0;
            for (int64_t idx = cluster_id; idx < p.items && ok; idx += nclusters, ++round) {
                const FwItem c = fw_decode_item(p, idx);
                const int64_t tt0 = c.band * p.band_tiles;
                const int64_t tt1 = tt0 + p.band_tiles < p.token_tiles ? tt0 + p.band_tiles : p.token_tiles;
                const int64_t left = p.items - round * nclusters;
                const int round_ctas = 2 * (int)(left < nclusters ? left : nclusters);
                const int b_row = (int)(c.ot * p.out_tile + rank * p.peer_row_offset);
                for (int64_t tt = tt0; tt < tt1 && ok; ++tt) {
                    {   // re-align with the other CTAs of this round (bounded: a late CTA just is not waited for)
                        const int t_in_item = (int)(tt - tt0);
                        const int target = (int)(round * gridDim.x) * p.band_tiles + round_ctas * (t_in_item + 1);
                        atomicAdd(p.align_counter, 1);
                        const unsigned long long t0 = global_ns();
                        while (*reinterpret_cast<volatile int *>(p.align_counter) < target && global_ns() - t0 < FW_ALIGN_NS) { }
                    }
                    const int a_row = (int)(tt * 2 * FW_BM + rank * FW_BM);
                    for (int64_t kb = 0; kb < p.k_blocks; ++kb) {
                        if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                        const uint32_t sbase = base + stage * FW_STAGE_BYTES;
                        const uint32_t fb = leader_full + 8 * stage;
                        if (rank == 0) mbar_arrive_expect_tx(bar_full + 8 * stage, 2 * FW_STAGE_BYTES);   // both CTAs' bytes
                        tma_load_2d_pair(sbase, &map_a, fb, (int)(kb * FW_BK), a_row, pol_a);
                        tma_load_2d_pair(sbase + FW_TILE_BYTES, map_b, fb, (int)(kb * FW_BK), b_row, pol_b);
                        if (++stage == FW_STAGES) { stage = 0; phase ^= 1u; }
                    }
                }
                // a short last band still counts band_tiles arrivals, so later rounds' targets hold
                if (tt1 - tt0 < p.band_tiles) atomicAdd(p.align_counter, (int)(p.band_tiles - (tt1 - tt0)));
            }
            if (!ok) { *abort_flag = 1; atomicExch(p.status, (int)DASS_ERR_TIMEOUT); }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = idesc_bf16_f32(2 * FW_BM, FW_BN);
            uint32_t stage = 0, phase = 0, tile = 0;
            bool ok = true;
            for (int64_t idx = cluster_id; idx < p.items && ok; idx += nclusters) {
                const FwItem c = fw_decode_item(p, idx);
                const int64_t tt0 = c.band * p.band_tiles;
                const int64_t tt1 = tt0 + p.band_tiles < p.token_tiles ? tt0 + p.band_tiles : p.token_tiles;
                for (int64_t tt = tt0; tt < tt1 && ok; ++tt, ++tile) {
                    // the epilogues of both CTAs must have drained this accumulator (two tiles ago)
                    const uint32_t as = tile & 1u;
                    if (!mbar_wait(bar_acc_empty + 8 * as, ((tile >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t acc_addr = tmem_base + as * FW_BN;
                    for (int64_t kb = 0; kb < p.k_blocks; ++kb) {
                        if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t sbase = base + stage * FW_STAGE_BYTES;
                        const uint64_t da = smem_desc_sw128(sbase);
                        const uint64_t db = smem_desc_sw128(sbase + FW_TILE_BYTES);
#pragma unroll
                        for (int k = 0; k < FW_BK / FW_UMMA_K; ++k) {
                            const uint32_t acc = (kb > 0 || k > 0) ? 1u : 0u;
                            const uint64_t koff = (uint64_t)(k * FW_UMMA_K * 2 / 16);   // 32 bytes per k step
                            umma_bf16_pair(acc_addr, da + koff, db + koff, idesc, acc);
                        }
                        umma_commit_pair(bar_empty + 8 * stage, (uint16_t)3);   // slot free in both CTAs
                        if (++stage == FW_STAGES) { stage = 0; phase ^= 1u; }
                    }
                    if (ok) umma_commit_pair(bar_acc_full + 8 * as, (uint16_t)3);   // accumulator ready in both CTAs
                }
            }
            if (!ok) { *abort_flag = 1; atomicExch(p.status, (int)DASS_ERR_TIMEOUT); }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue (4 warps, this CTA's 128 tokens)
        const int quad = warp & 3;                               // TMEM lanes 32*quad .. 32*quad+31
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        const uint32_t leader_acc_empty = map_to_cta(bar_acc_empty, 0);
        uint32_t tile = 0;
        bool ok = true;
        for (int64_t idx = cluster_id; idx < p.items && ok; idx += nclusters) {
            const FwItem c = fw_decode_item(p, idx);
            const int64_t tt0 = c.band * p.band_tiles;
            const int64_t tt1 = tt0 + p.band_tiles < p.token_tiles ? tt0 + p.band_tiles : p.token_tiles;
            const int64_t n_base = c.ot * p.out_tile;            // first output column of this item
            for (int64_t tt = tt0; tt < tt1 && ok; ++tt, ++tile) {
                const uint32_t as = tile & 1u;
                if (!mbar_wait(bar_acc_full + 8 * as, (tile >> 1) & 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const int64_t t = tt * 2 * FW_BM + rank * FW_BM + quad * 32 + lane;   // this thread's token
                uint16_t *row = p.out + (t < p.T ? t : 0) * p.ldo;
                const uint32_t acc_addr = lane_addr + as * FW_BN;
                if constexpr (MODE == MODE_GLU) {
#pragma unroll 1
                    for (int col = 0; col < FW_BN / 2; col += 32) {
                        uint32_t g[32], u[32], w[16];
                        tmem_ld_32(acc_addr + col, g);
                        tmem_ld_32(acc_addr + FW_BN / 2 + col, u);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            w[j] = fw_pack_bf16(glu_h<ACT>(__uint_as_float(g[2 * j]), __uint_as_float(u[2 * j])),
                                                glu_h<ACT>(__uint_as_float(g[2 * j + 1]), __uint_as_float(u[2 * j + 1])));
                        if (t < p.T) fw_store_32(p, row, n_base + col, w);
                    }
                } else {
#pragma unroll 1
                    for (int col = 0; col < FW_BN; col += 32) {
                        uint32_t a[32], w[16];
                        tmem_ld_32(acc_addr + col, a);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; ++j) w[j] = fw_pack_bf16(__uint_as_float(a[2 * j]), __uint_as_float(a[2 * j + 1]));
                        if (t < p.T) fw_store_32(p, row, n_base + col, w);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {                                 // release the accumulator to the leader's MMA warp
                    if (rank == 0) mbar_arrive(bar_acc_empty + 8 * as);
                    else mbar_arrive_cluster(leader_acc_empty + 8 * as);
                }
            }
        }
        if (!ok && lane == 0) { *abort_flag = 1; atomicExch(p.status, (int)DASS_ERR_TIMEOUT); }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // failure path only: give copies and MMAs that were already issued time to land before the
        // shared memory and the TMEM columns are handed back
        for (int i = 0; i < 20; ++i) __nanosleep(1000000);
        __syncthreads();
    }
    cluster_sync_all();            // the peer no longer signals into this CTA's shared memory or uses the pair's TMEM
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, FW_TMEM_COLS);
    }
}

// ------------------------------------------------------------------ host side
bool tc_make_map(CUtensorMap *map, const void *ptr, int64_t rows, int64_t cols, int64_t ld, int box_rows);   // calib_tc.cu
int device_sm_count();                                                                                       // dass_abi.cu

__global__ void fw_counters_clear_kernel(int *words)
{
    if (threadIdx.x == 0) { words[1] = 0; words[2] = 0; }
}

cudaError_t mlp_forward_counters_clear(int *words, cudaStream_t st)
{
    fw_counters_clear_kernel<<<1, 32, 0, st>>>(words);
    return cudaGetLastError();
}

// Token tiles per band: as many as 16 (a right-operand tile then serves 16 token tiles from L2), fewer when that
// would leave the persistent grid with only a handful of rounds and a long idle tail.
static int fw_pick_band_tiles(int64_t out_tiles, int64_t token_tiles, int pairs)
{
    for (int bt = 16; bt > 1; bt >>= 1) {
        const int64_t bands = (token_tiles + bt - 1) / bt;
        if (out_tiles * bands >= 12ll * pairs) return bt;
    }
    return 1;
}

template <int MODE, int ACT>
static cudaError_t fw_launch(const CUtensorMap &ma, const CUtensorMap &mb0, const CUtensorMap &mb1, const FwParams &p,
                             int grid, cudaStream_t st)
{
    static DeviceMask configured{0ull};               // per device
    const cudaError_t ce = ensure_dynamic_smem(mlp_forward_tc_kernel<MODE, ACT>, (int)FW_SMEM_BYTES, configured);
    if (ce != cudaSuccess) return ce;
    mlp_forward_tc_kernel<MODE, ACT><<<grid, FW_THREADS, FW_SMEM_BYTES, st>>>(ma, mb0, mb1, p);
    return cudaGetLastError();
}

static int fw_fill_items(FwParams &p, int64_t n_out, int64_t T, int64_t k)
{
    const int pairs = device_sm_count() / 2;
    p.out_tiles = (n_out + p.out_tile - 1) / p.out_tile;
    p.token_tiles = (T + 2 * FW_BM - 1) / (2 * FW_BM);
    p.band_tiles = fw_pick_band_tiles(p.out_tiles, p.token_tiles, pairs);
    p.bands = (p.token_tiles + p.band_tiles - 1) / p.band_tiles;
    p.items = p.out_tiles * p.bands;
    p.k_blocks = (k + FW_BK - 1) / FW_BK;
    p.vector_ok = ((reinterpret_cast<uintptr_t>(p.out) & 15u) == 0 && p.ldo % 8 == 0) ? 1 : 0;
    return 2 * (int)(p.items < pairs ? p.items : pairs);        // CTAs: whole pairs
}

// One chunk of tokens: H[T x I] = Eq. 2 (pitch ldh), then Z[T x d] = Eq. 3.  `words` = {status, counter, counter}.
dass_status mlp_forward_tc_launch(const void *X, int64_t T, int64_t ldx, const void *Wg, const void *Wu,
                                  int64_t I, int64_t d, int64_t ldw, const void *Wd, int64_t ldd, int act,
                                  void *H, int64_t ldh, void *Z, int64_t ldz, int *words, cudaStream_t st)
{
    const int64_t lim = 0x7fffffffll - 512;
    if (d > lim || T > lim || I > lim) return DASS_ERR_UNSUPPORTED;
    if (device_sm_count() < 2) return DASS_ERR_UNSUPPORTED;
    CUtensorMap mx, mg, mu, mh, md;
    if (!tc_make_map(&mx, X, T, d, ldx, FW_BM) || !tc_make_map(&mg, Wg, I, d, ldw, 128) ||
        !tc_make_map(&mu, Wu, I, d, ldw, 128) || !tc_make_map(&mh, H, T, I, ldh, FW_BM) ||
        !tc_make_map(&md, Wd, d, I, ldd, 128))
        return DASS_ERR_CUDA;

    FwParams pg;
    pg.out = static_cast<uint16_t *>(H); pg.ldo = ldh;
    pg.status = words; pg.align_counter = words + 1;
    pg.T = T; pg.n_out = I; pg.out_tile = FW_BN / 2; pg.peer_row_offset = 0;
    pg.super_bands = 16;
    const int grid_g = fw_fill_items(pg, I, T, d);
    cudaError_t e;
    switch (act) {
    case DASS_ACT_SILU: e = fw_launch<MODE_GLU, DASS_ACT_SILU>(mx, mg, mu, pg, grid_g, st); break;
    case DASS_ACT_GELU_TANH: e = fw_launch<MODE_GLU, DASS_ACT_GELU_TANH>(mx, mg, mu, pg, grid_g, st); break;
    default: e = fw_launch<MODE_GLU, DASS_ACT_RELU>(mx, mg, mu, pg, grid_g, st); break;
    }
    if (e != cudaSuccess) return DASS_ERR_CUDA;

    FwParams pd;
    pd.out = static_cast<uint16_t *>(Z); pd.ldo = ldz;
    pd.status = words; pd.align_counter = words + 2;
    pd.T = T; pd.n_out = d; pd.out_tile = FW_BN; pd.peer_row_offset = FW_BN / 2;
    pd.super_bands = 8;      // the contraction runs over I: operand tiles are too large to stay in L2, so the pairs
                             // running together form a squarer patch of output tiles (8 bands x ~9 output tiles)
    const int grid_d = fw_fill_items(pd, d, T, I);
    e = fw_launch<MODE_PLAIN, DASS_ACT_SILU>(mh, md, md, pd, grid_d, st);
    return e == cudaSuccess ? DASS_OK : DASS_ERR_CUDA;
}

}  // namespace dass
