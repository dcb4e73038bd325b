// Forward pass of the (pruned) GLU MLP layer for bf16 tensors, Eq. 2 then Eq. 3, on the sm_100a tensor cores:
//
//   kernel <MODE_GLU>    H[t, i] = bf16( act(x_t . Wg_i) * (x_t . Wu_i) )          (Eq. 2)
//   kernel <MODE_PLAIN>  Z[t, n] = bf16( h_t . Wd_n )                               (Eq. 3)
//
// Both are the same persistent, warp-specialised kernel: two 128-row A tiles (gate and up rows of the
// same neurons; or two consecutive 128-row blocks of Wd) share one 256-token B tile, accumulate in two
// 128 x 256 fp32 TMEM blocks, and an epilogue thread per A row (TMEM lane) turns its 256 token columns into
// bf16 outputs.  Pruned weights are zeros stored in place, so the dense contraction is the pruned layer.
//   warp 0      TMA producer into a 3-stage, 128B-swizzled shared-memory ring
//   warp 1      allocates TMEM, issues tcgen05.mma (one lane), commits ring slots and accumulators
//   warps 2..5  epilogue: tcgen05.ld, activation and gating product (MODE_GLU), round to bf16, store
// Work items are (A tile, band of token tiles), ordered so that the CTAs running together share a few A
// and B tiles through L2; the producers re-align at tile boundaries with a bounded counting barrier, A
// loads are evict-last and B loads evict-first, as in the calibration kernel.
//
// Every wait on an mbarrier is bounded: when one runs out the CTA raises an abort flag, records
// DASS_ERR_TIMEOUT in the status word, lets its roles drain and frees its TMEM before returning.
#include "tc_common.cuh"

namespace dass {

constexpr int FW_BM = 128;         // A rows per accumulator (MMA M, TMEM lanes)
constexpr int FW_BN = 256;         // tokens per tile (MMA N)
constexpr int FW_BK = 64;          // k per ring slot: 64 bf16 = one 128-byte swizzle row
constexpr int FW_UMMA_K = 16;
constexpr int FW_STAGES = 3;
constexpr int FW_SUPER_BANDS = 16;   // bands interleaved in the item order for L2 sharing
constexpr unsigned long long FW_ALIGN_NS = 20000ull;
constexpr int FW_THREADS = 192;
constexpr uint32_t FW_A_BYTES = FW_BM * FW_BK * 2;                 // 16 KB
constexpr uint32_t FW_B_BYTES = FW_BN * FW_BK * 2;                 // 32 KB
constexpr uint32_t FW_STAGE_BYTES = 2 * FW_A_BYTES + FW_B_BYTES;   // 64 KB
constexpr uint32_t FW_TMEM_COLS = 512;
constexpr uint32_t FW_SMEM_BYTES = FW_STAGES * FW_STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;

constexpr int MODE_GLU = 0, MODE_PLAIN = 1;

struct FwParams {
    uint16_t *out;        // [T x n_out] bf16, pitch ldo
    int64_t ldo;
    int *status;          // device status word (0 = ok)
    int *align_counter;   // arrivals of the tile-boundary alignment barrier (zero before the launch)
    int64_t T;            // tokens
    int64_t n_out;        // output columns: I (MODE_GLU) or d (MODE_PLAIN)
    int64_t a_tile_rows;  // A rows (= output columns) per item: 128 (MODE_GLU) or 256 (MODE_PLAIN)
    int64_t a1_offset;    // row offset of the second A tile inside its tensor map: 0 or 128
    int64_t a_tiles, token_tiles, bands, items, k_blocks;
    int band_tiles;       // token tiles per band
};

struct FwItem { int64_t at, band; };

__device__ __forceinline__ FwItem fw_decode_item(const FwParams &p, int64_t idx)
{
    const int64_t per_super = p.a_tiles * FW_SUPER_BANDS;
    const int64_t sb = idx / per_super;
    const int64_t rem = idx - sb * per_super;
    const int64_t left = p.bands - sb * FW_SUPER_BANDS;
    const int64_t nb = left < FW_SUPER_BANDS ? left : FW_SUPER_BANDS;
    FwItem c;
    c.at = rem / nb;
    c.band = sb * FW_SUPER_BANDS + (rem - c.at * nb);
    return c;
}

__device__ __forceinline__ uint16_t fw_to_bf16(float v)
{
    uint16_t r;
    asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(r) : "f"(v));
    return r;
}

template <int MODE, int ACT>
__global__ void __launch_bounds__(FW_THREADS, 1)
mlp_forward_tc_kernel(const __grid_constant__ CUtensorMap map_b, const __grid_constant__ CUtensorMap map_a0,
                      const __grid_constant__ CUtensorMap map_a1, const FwParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;                 // swizzled tiles need 1024-byte alignment
    uint8_t *aligned = smem_raw + (base - raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(aligned + FW_STAGES * FW_STAGE_BYTES);
    const uint32_t bar_full = smem_u32(bars);                     // [FW_STAGES]
    const uint32_t bar_empty = bar_full + 8 * FW_STAGES;          // [FW_STAGES]
    const uint32_t bar_acc_full = bar_empty + 8 * FW_STAGES;
    const uint32_t bar_acc_empty = bar_acc_full + 8;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * FW_STAGES + 2);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < FW_STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_acc_full, 1);
        mbar_init(bar_acc_empty, 4);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), FW_TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            // an A tile is re-read for every token tile of a band: keep it in L2; a B tile is shared only by
            // the CTAs reading it right now: let it go first
            const uint64_t pol_a = l2_policy_evict_last();
            const uint64_t pol_b = l2_policy_evict_first();
            int64_t round = 0;
            for (int64_t idx = blockIdx.x; idx < p.items && ok; idx += gridDim.x, ++round) {
                const FwItem c = fw_decode_item(p, idx);
                const int64_t tt0 = c.band * p.band_tiles;
                const int64_t tt1 = tt0 + p.band_tiles < p.token_tiles ? tt0 + p.band_tiles : p.token_tiles;
                const int64_t left = p.items - round * gridDim.x;
                const int round_ctas = (int)(left < (int64_t)gridDim.x ? left : (int64_t)gridDim.x);
                const int a_row = (int)(c.at * p.a_tile_rows);
                for (int64_t tt = tt0; tt < tt1 && ok; ++tt) {
                    // re-align with the other CTAs of this round (bounded: a late CTA just is not waited for)
                    {
                        const int t_in_item = (int)(tt - tt0);
                        const int target = (int)(round * gridDim.x) * p.band_tiles + round_ctas * (t_in_item + 1);
                        atomicAdd(p.align_counter, 1);
                        const unsigned long long t0 = global_ns();
                        while (*reinterpret_cast<volatile int *>(p.align_counter) < target && global_ns() - t0 < FW_ALIGN_NS) { }
                    }
                    for (int64_t kb = 0; kb < p.k_blocks; ++kb) {
                        if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                        const uint32_t sbase = base + stage * FW_STAGE_BYTES;
                        const uint32_t fb = bar_full + 8 * stage;
                        mbar_arrive_expect_tx(fb, FW_STAGE_BYTES);
                        tma_load_2d_hint(sbase, &map_a0, fb, (int)(kb * FW_BK), a_row, pol_a);
                        tma_load_2d_hint(sbase + FW_A_BYTES, &map_a1, fb, (int)(kb * FW_BK), a_row + (int)p.a1_offset, pol_a);
                        tma_load_2d_hint(sbase + 2 * FW_A_BYTES, &map_b, fb, (int)(kb * FW_BK), (int)(tt * FW_BN), pol_b);
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
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16_f32(FW_BM, FW_BN);
            uint32_t stage = 0, phase = 0, tile = 0;
            bool ok = true;
            for (int64_t idx = blockIdx.x; idx < p.items && ok; idx += gridDim.x) {
                const FwItem c = fw_decode_item(p, idx);
                const int64_t tt0 = c.band * p.band_tiles;
                const int64_t tt1 = tt0 + p.band_tiles < p.token_tiles ? tt0 + p.band_tiles : p.token_tiles;
                for (int64_t tt = tt0; tt < tt1 && ok; ++tt, ++tile) {
                    // the epilogue must have drained the previous tile's accumulators
                    if (!mbar_wait(bar_acc_empty, (tile & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    for (int64_t kb = 0; kb < p.k_blocks; ++kb) {
                        if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t sbase = base + stage * FW_STAGE_BYTES;
                        const uint64_t da0 = smem_desc_sw128(sbase);
                        const uint64_t da1 = smem_desc_sw128(sbase + FW_A_BYTES);
                        const uint64_t db = smem_desc_sw128(sbase + 2 * FW_A_BYTES);
#pragma unroll
                        for (int k = 0; k < FW_BK / FW_UMMA_K; ++k) {
                            const uint32_t acc = (kb > 0 || k > 0) ? 1u : 0u;
                            const uint64_t koff = (uint64_t)(k * FW_UMMA_K * 2 / 16);   // 32 bytes per k step
                            umma_bf16(tmem_base, da0 + koff, db + koff, idesc, acc);
                            umma_bf16(tmem_base + FW_BN, da1 + koff, db + koff, idesc, acc);
                        }
                        umma_commit(bar_empty + 8 * stage);      // slot reusable once these MMAs have read it
                        if (++stage == FW_STAGES) { stage = 0; phase ^= 1u; }
                    }
                    if (ok) umma_commit(bar_acc_full);            // accumulators complete
                }
            }
            if (!ok) { *abort_flag = 1; atomicExch(p.status, (int)DASS_ERR_TIMEOUT); }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue (4 warps, 128 A rows)
        const int quad = warp & 3;                               // TMEM lanes 32*quad .. 32*quad+31
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        uint32_t tile = 0;
        bool ok = true;
        for (int64_t idx = blockIdx.x; idx < p.items && ok; idx += gridDim.x) {
            const FwItem c = fw_decode_item(p, idx);
            const int64_t tt0 = c.band * p.band_tiles;
            const int64_t tt1 = tt0 + p.band_tiles < p.token_tiles ? tt0 + p.band_tiles : p.token_tiles;
            // output column(s) of this thread: one per accumulator row it owns
            const int64_t n0 = c.at * p.a_tile_rows + quad * 32 + lane;
            const int64_t n1 = n0 + FW_BM;                       // MODE_PLAIN only
            const bool n0_ok = n0 < p.n_out;
            const bool n1_ok = MODE == MODE_PLAIN && n1 < p.n_out;
            for (int64_t tt = tt0; tt < tt1 && ok; ++tt, ++tile) {
                if (!mbar_wait(bar_acc_full, tile & 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const int64_t t_base = tt * FW_BN;
                const int64_t t_left = p.T - t_base;
                const int valid = (int)(t_left < FW_BN ? t_left : FW_BN);       // tokens of this tile that exist
#pragma unroll 1
                for (int col = 0; col < FW_BN; col += 32) {
                    uint32_t g[32], u[32];
                    tmem_ld_32(lane_addr + col, g);
                    tmem_ld_32(lane_addr + FW_BN + col, u);
                    tmem_wait_ld();
                    uint16_t *dst = p.out + (t_base + col) * p.ldo;
                    const int nj = valid - col;                                 // tokens of this block that exist (may be <= 0)
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        if (j < nj) {
                            if constexpr (MODE == MODE_GLU) {
                                const float h = glu_h<ACT>(__uint_as_float(g[j]), __uint_as_float(u[j]));
                                if (n0_ok) dst[j * p.ldo + n0] = fw_to_bf16(h);
                            } else {
                                if (n0_ok) dst[j * p.ldo + n0] = fw_to_bf16(__uint_as_float(g[j]));
                                if (n1_ok) dst[j * p.ldo + n1] = fw_to_bf16(__uint_as_float(u[j]));
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_acc_empty);
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
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, FW_TMEM_COLS);
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

// Token tiles per band: as many as 16 (an A tile then serves 16 token tiles from L2), fewer when that would
// leave the persistent grid with only a handful of rounds and a long idle tail.
static int fw_pick_band_tiles(int64_t a_tiles, int64_t token_tiles, int grid_cap)
{
    for (int bt = 16; bt > 1; bt >>= 1) {
        const int64_t bands = (token_tiles + bt - 1) / bt;
        if (a_tiles * bands >= 12ll * grid_cap) return bt;
    }
    return 1;
}

template <int MODE, int ACT>
static cudaError_t fw_launch(const CUtensorMap &mb, const CUtensorMap &ma0, const CUtensorMap &ma1, const FwParams &p,
                             int grid, cudaStream_t st)
{
    static bool configured = false;
    if (!configured) {
        const cudaError_t e = cudaFuncSetAttribute(mlp_forward_tc_kernel<MODE, ACT>,
                                                   cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FW_SMEM_BYTES);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    mlp_forward_tc_kernel<MODE, ACT><<<grid, FW_THREADS, FW_SMEM_BYTES, st>>>(mb, ma0, ma1, p);
    return cudaGetLastError();
}

static void fw_fill_items(FwParams &p, int64_t a_rows, int64_t T, int64_t k)
{
    p.a_tiles = (a_rows + p.a_tile_rows - 1) / p.a_tile_rows;
    p.token_tiles = (T + FW_BN - 1) / FW_BN;
    p.band_tiles = fw_pick_band_tiles(p.a_tiles, p.token_tiles, device_sm_count());
    p.bands = (p.token_tiles + p.band_tiles - 1) / p.band_tiles;
    p.items = p.a_tiles * p.bands;
    p.k_blocks = (k + FW_BK - 1) / FW_BK;
}

// One chunk of tokens: H[T x I] = Eq. 2 (pitch ldh), then Z[T x d] = Eq. 3.  `words` = {status, counter, counter}.
dass_status mlp_forward_tc_launch(const void *X, int64_t T, int64_t ldx, const void *Wg, const void *Wu,
                                  int64_t I, int64_t d, int64_t ldw, const void *Wd, int64_t ldd, int act,
                                  void *H, int64_t ldh, void *Z, int64_t ldz, int *words, cudaStream_t st)
{
    const int64_t lim = 0x7fffffffll - 512;
    if (d > lim || T > lim || I > lim) return DASS_ERR_UNSUPPORTED;
    CUtensorMap mx, mg, mu, mh, md;
    if (!tc_make_map(&mx, X, T, d, ldx, FW_BN) || !tc_make_map(&mg, Wg, I, d, ldw, FW_BM) ||
        !tc_make_map(&mu, Wu, I, d, ldw, FW_BM) || !tc_make_map(&mh, H, T, I, ldh, FW_BN) ||
        !tc_make_map(&md, Wd, d, I, ldd, FW_BM))
        return DASS_ERR_CUDA;
    const int sms = device_sm_count();

    FwParams pg;
    pg.out = static_cast<uint16_t *>(H); pg.ldo = ldh;
    pg.status = words; pg.align_counter = words + 1;
    pg.T = T; pg.n_out = I; pg.a_tile_rows = FW_BM; pg.a1_offset = 0;
    fw_fill_items(pg, I, T, d);
    const int grid_g = (int)(pg.items < sms ? pg.items : sms);
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
    pd.T = T; pd.n_out = d; pd.a_tile_rows = 2 * FW_BM; pd.a1_offset = FW_BM;
    fw_fill_items(pd, d, T, I);
    const int grid_d = (int)(pd.items < sms ? pd.items : sms);
    e = fw_launch<MODE_PLAIN, DASS_ACT_SILU>(mh, md, md, pd, grid_d, st);
    return e == cudaSuccess ? DASS_OK : DASS_ERR_CUDA;
}

}  // namespace dass
