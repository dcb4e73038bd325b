// Stage (a) for bf16 inputs: Eq. 2 and the per-neuron sum of squares on the sm_100a tensor cores.
//
//   G = Wg_tile . X_tile^T,  U = Wu_tile . X_tile^T      (tcgen05.mma, bf16 x bf16 -> fp32 in TMEM)
//   sumsq[neuron] += sum over the tile's tokens of ( act(G) * U )^2                (fused epilogue)
//
// Neurons are the MMA M dimension (128 per tile = the 128 TMEM lanes), tokens the N dimension (256
// per tile), so one epilogue thread owns one neuron and adds up its tokens serially in registers --
// no shuffles, no atomics -- and the intermediate activation H never reaches memory.  The gate and up
// tiles are two A operands that share one B operand (the X tile).
//
// One persistent CTA per SM, warp-specialised:
//   warp 0      TMA producer: X / Wg / Wu k-slices into a 3-stage, 128B-swizzled shared-memory ring
//   warp 1      allocates TMEM, issues the MMAs (one lane), commits ring slots and accumulators
//   warps 2..5  epilogue: tcgen05.ld the two accumulators, activation, gating product, square, sum
// A work item is (neuron tile, band of up to 16 token tiles); items are ordered so that the CTAs
// running at the same moment share a few X tiles and a few W tiles through L2.  That sharing only works
// while those CTAs read the same k-slices at about the same time, so the producers re-align at every tile
// boundary (a counting barrier on a global word with a 20 us bound), W loads carry an L2 evict-last
// policy (a W tile is re-read for each of the band's token tiles) and X loads evict-first.  Measured on
// the 70B-shaped layer this cut DRAM reads 2.5x.  Every item writes one partial per neuron to
// partial[band][neuron]; a second tiny kernel adds the bands in a fixed order.
//
// Every wait on an mbarrier is bounded: when a wait runs out the CTA raises an abort flag, records
// DASS_ERR_TIMEOUT in the status word, lets its roles drain and frees its TMEM before returning.
#include "tc_common.cuh"

namespace dass {

constexpr int TC_BM = 128;         // neurons per tile (MMA M, TMEM lanes)
constexpr int TC_BN = 256;         // tokens per tile (MMA N)
constexpr int TC_BK = 64;          // k per ring slot: 64 bf16 = one 128-byte swizzle row
constexpr int TC_UMMA_K = 16;      // k per tcgen05.mma for 16-bit inputs
constexpr int TC_STAGES = 3;
constexpr int TC_MAX_BAND_TILES = 16;   // token tiles per band (one partial per band and neuron) at most
constexpr int TC_SUPER_BANDS = 16;   // bands interleaved in the item order for L2 sharing, at most
constexpr unsigned long long TC_ALIGN_NS = 20000ull;   // longest a CTA waits for the others at a tile boundary
constexpr int TC_THREADS = 192;
constexpr uint32_t TC_W_BYTES = TC_BM * TC_BK * 2;                 // 16 KB
constexpr uint32_t TC_X_BYTES = TC_BN * TC_BK * 2;                 // 32 KB
constexpr uint32_t TC_STAGE_BYTES = 2 * TC_W_BYTES + TC_X_BYTES;   // 64 KB
constexpr uint32_t TC_TMEM_COLS = 512;                             // G: columns 0..255, U: 256..511
constexpr uint32_t TC_SMEM_BYTES = TC_STAGES * TC_STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;

struct TcParams {
    double *partial;     // [bands][I]
    int *status;         // device status word (0 = ok)
    int *align_counter;  // arrivals of the tile-boundary alignment barrier (zeroed before the launch)
    int64_t T, I, d;
    int64_t neuron_tiles, token_tiles, bands, items, k_blocks;
    int band_tiles;      // token tiles per band (calib_tc_band_tiles)
    int super_bands;     // bands interleaved in the item order (calib_tc_super_bands)
};

struct ItemCoord { int64_t nt, band; };

__device__ __forceinline__ ItemCoord decode_item(const TcParams &p, int64_t idx)
{
    const int64_t per_super = p.neuron_tiles * p.super_bands;
    const int64_t sb = idx / per_super;
    const int64_t rem = idx - sb * per_super;
    const int64_t left = p.bands - sb * p.super_bands;
    const int64_t nb = left < p.super_bands ? left : p.super_bands;
    ItemCoord c;
    c.nt = rem / nb;
    c.band = sb * p.super_bands + (rem - c.nt * nb);
    return c;
}

template <int ACT>
__global__ void __launch_bounds__(TC_THREADS, 1)
calib_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_wg,
                const __grid_constant__ CUtensorMap map_wu, const TcParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;                 // swizzled tiles need 1024-byte alignment
    uint8_t *aligned = smem_raw + (base - raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(aligned + TC_STAGES * TC_STAGE_BYTES);
    const uint32_t bar_full = smem_u32(bars);                     // [TC_STAGES]
    const uint32_t bar_empty = bar_full + 8 * TC_STAGES;          // [TC_STAGES]
    const uint32_t bar_acc_full = bar_empty + 8 * TC_STAGES;
    const uint32_t bar_acc_empty = bar_acc_full + 8;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * TC_STAGES + 2);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < TC_STAGES; ++s) {
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
        tmem_alloc(smem_u32(tmem_slot), TC_TMEM_COLS);
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
            // W tiles are re-read for every token tile of a band: keep them in L2; X tiles are shared only
            // by the CTAs reading them right now: let them go first.
            const uint64_t pol_w = l2_policy_evict_last();
            const uint64_t pol_x = l2_policy_evict_first();
            int64_t round = 0;
            for (int64_t idx = blockIdx.x; idx < p.items && ok; idx += gridDim.x, ++round) {
                const ItemCoord c = decode_item(p, idx);
                const int64_t tt0 = c.band * p.band_tiles;
                const int64_t tt1 = tt0 + p.band_tiles < p.token_tiles ? tt0 + p.band_tiles : p.token_tiles;
                const int64_t left = p.items - round * gridDim.x;
                const int round_ctas = (int)(left < (int64_t)gridDim.x ? left : (int64_t)gridDim.x);   // CTAs with an item in this round
                for (int64_t tt = tt0; tt < tt1 && ok; ++tt) {
                    // Re-align with the other CTAs of this round before loading the tile: the CTAs that
                    // run together share X and W tiles through L2 only while they read the same k-slices
                    // at about the same time.  A counting barrier on a global word, never waited on for
                    // longer than TC_ALIGN_NS (a late or absent CTA just is not waited for).
                    {
                        const int t_in_item = (int)(tt - tt0);
                        const int target = (int)(round * gridDim.x) * p.band_tiles + round_ctas * (t_in_item + 1);
                        atomicAdd(p.align_counter, 1);
                        const unsigned long long t0 = global_ns();
                        while (*reinterpret_cast<volatile int *>(p.align_counter) < target && global_ns() - t0 < TC_ALIGN_NS) { }
                    }
                    for (int64_t kb = 0; kb < p.k_blocks; ++kb) {
                        if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                        const uint32_t sbase = base + stage * TC_STAGE_BYTES;
                        const uint32_t fb = bar_full + 8 * stage;
                        mbar_arrive_expect_tx(fb, TC_STAGE_BYTES);
                        tma_load_2d_hint(sbase, &map_wg, fb, (int)(kb * TC_BK), (int)(c.nt * TC_BM), pol_w);
                        tma_load_2d_hint(sbase + TC_W_BYTES, &map_wu, fb, (int)(kb * TC_BK), (int)(c.nt * TC_BM), pol_w);
                        tma_load_2d_hint(sbase + 2 * TC_W_BYTES, &map_x, fb, (int)(kb * TC_BK), (int)(tt * TC_BN), pol_x);
                        if (++stage == TC_STAGES) { stage = 0; phase ^= 1u; }
                    }
                }
                // a short last band still counts p.band_tiles arrivals, so later rounds' targets hold
                if (tt1 - tt0 < p.band_tiles) atomicAdd(p.align_counter, (int)(p.band_tiles - (tt1 - tt0)));
            }
            if (!ok) { *abort_flag = 1; atomicExch(p.status, (int)DASS_ERR_TIMEOUT); }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16_f32(TC_BM, TC_BN);
            uint32_t stage = 0, phase = 0, tile = 0;
            bool ok = true;
            for (int64_t idx = blockIdx.x; idx < p.items && ok; idx += gridDim.x) {
                const ItemCoord c = decode_item(p, idx);
                const int64_t tt0 = c.band * p.band_tiles;
                const int64_t tt1 = tt0 + p.band_tiles < p.token_tiles ? tt0 + p.band_tiles : p.token_tiles;
                for (int64_t tt = tt0; tt < tt1 && ok; ++tt, ++tile) {
                    // the epilogue must have drained the previous tile's accumulators
                    if (!mbar_wait(bar_acc_empty, (tile & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    for (int64_t kb = 0; kb < p.k_blocks; ++kb) {
                        if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t sbase = base + stage * TC_STAGE_BYTES;
                        const uint64_t dg = smem_desc_sw128(sbase);
                        const uint64_t du = smem_desc_sw128(sbase + TC_W_BYTES);
                        const uint64_t dx = smem_desc_sw128(sbase + 2 * TC_W_BYTES);
#pragma unroll
                        for (int k = 0; k < TC_BK / TC_UMMA_K; ++k) {
                            const uint32_t acc = (kb > 0 || k > 0) ? 1u : 0u;
                            const uint64_t koff = (uint64_t)(k * TC_UMMA_K * 2 / 16);   // 32 bytes per k step
                            umma_bf16(tmem_base, dg + koff, dx + koff, idesc, acc);
                            umma_bf16(tmem_base + TC_BN, du + koff, dx + koff, idesc, acc);
                        }
                        umma_commit(bar_empty + 8 * stage);      // slot reusable once these MMAs have read it
                        if (++stage == TC_STAGES) { stage = 0; phase ^= 1u; }
                    }
                    if (ok) umma_commit(bar_acc_full);            // accumulators complete
                }
            }
            if (!ok) { *abort_flag = 1; atomicExch(p.status, (int)DASS_ERR_TIMEOUT); }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue (4 warps, 128 neurons)
        const int quad = warp & 3;                               // TMEM lanes 32*quad .. 32*quad+31
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        uint32_t tile = 0;
        bool ok = true;
        for (int64_t idx = blockIdx.x; idx < p.items && ok; idx += gridDim.x) {
            const ItemCoord c = decode_item(p, idx);
            const int64_t tt0 = c.band * p.band_tiles;
            const int64_t tt1 = tt0 + p.band_tiles < p.token_tiles ? tt0 + p.band_tiles : p.token_tiles;
            double acc = 0.0;
            for (int64_t tt = tt0; tt < tt1 && ok; ++tt, ++tile) {
                if (!mbar_wait(bar_acc_full, tile & 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                float s = 0.0f;
#pragma unroll 1
                for (int col = 0; col < TC_BN; col += 32) {
                    uint32_t g[32], u[32];
                    tmem_ld_32(lane_addr + col, g);
                    tmem_ld_32(lane_addr + TC_BN + col, u);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const float h = glu_h<ACT>(__uint_as_float(g[j]), __uint_as_float(u[j]));
                        s = fmaf(h, h, s);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_acc_empty);
                acc += (double)s;       // tokens past T are zero rows of X: act(0) * 0 adds nothing
            }
            const int64_t neuron = c.nt * TC_BM + quad * 32 + lane;
            if (ok && neuron < p.I) DASS_ST(&p.partial[c.band * p.I + neuron], acc);
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
        tmem_dealloc(tmem_base, TC_TMEM_COLS);
    }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn()
{
    static std::atomic<EncodeTiledFn> cached{nullptr};      // the same value whichever host thread resolves it first
    EncodeTiledFn fn = cached.load(std::memory_order_acquire);
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(ptr);
        cached.store(fn, std::memory_order_release);
    }
    return fn;
}

// Row-major bf16 matrix [rows x cols] with pitch ld: dimension 0 = the contiguous k axis.  Boxes are
// 64 x box_rows elements with the 128-byte swizzle; out-of-range elements read as zero.
bool tc_make_map(CUtensorMap *map, const void *ptr, int64_t rows, int64_t cols, int64_t ld, int box_rows)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)TC_BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Row-major bf16 matrix [rows x cols] with pitch ld, plain (un-swizzled) boxes of box_cols x box_rows elements;
// out-of-range elements read as zero.  Used by the streaming stage-(b) kernels.
bool tile_map_bf16(CUtensorMap *map, const void *ptr, int64_t rows, int64_t cols, int64_t ld, int box_cols, int box_rows)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int device_sm_count();   // dass_abi.cu

// Token tiles per band.  16 keeps a W tile in L2 for 16 token tiles; with few tokens that leaves the persistent
// grid (one CTA per SM: 148 on the B200 this library is written for) with a part-filled last round, so a shorter band is taken
// when it saves at least 1 % of the modelled time -- rounds x (band's k-blocks + a per-item cost of about 29
// k-blocks: new W tiles and the re-alignment of the CTAs, fitted to measurements) -- and the partial sums (one
// double per band and neuron) stay within 14 MiB and within `partial_budget_bytes`, what the caller's scratch has
// room for.  Bands of 16 are the fallback, so a scratch sized by the query for some token count also serves every
// shorter batch.  The entry points choose the band length and hand it to the launchers and to the reduction.
int calib_tc_band_tiles(int64_t T, int64_t I, int64_t d, int64_t partial_budget_bytes)
{
    const int64_t tiles = (I + TC_BM - 1) / TC_BM;
    const int64_t token_tiles = (T + TC_BN - 1) / TC_BN;
    const int64_t k_blocks = (d + TC_BK - 1) / TC_BK;
    auto bands = [&](int bt) { return (token_tiles + bt - 1) / bt; };
    const int64_t sms = device_sm_count();   // 148 when no device is current (the size query works without one)
    auto cost = [&](int bt) { return ((tiles * bands(bt) + sms - 1) / sms) * (bt * k_blocks + 29); };
    int best = TC_MAX_BAND_TILES;
    int64_t best_cost = cost(best);
    for (int bt = TC_MAX_BAND_TILES / 2; bt >= 1; bt >>= 1) {
        const int64_t bytes = bands(bt) * I * (int64_t)sizeof(double);
        if (bytes > ((int64_t)14 << 20) || bytes > partial_budget_bytes) break;
        const int64_t ct = cost(bt);
        if (ct * 100 < best_cost * 99) { best = bt; best_cost = ct; }
    }
    return best;
}

// Partial sums per neuron (= bands) for a band length.
int64_t calib_tc_parts_for(int64_t T, int band_tiles)
{
    const int64_t token_tiles = (T + TC_BN - 1) / TC_BN;
    return (token_tiles + band_tiles - 1) / band_tiles;
}

// The workspace query's answer: the preferred band length with no limit from the caller.
int64_t calib_tc_parts(int64_t T, int64_t I, int64_t d)
{
    return calib_tc_parts_for(T, calib_tc_band_tiles(T, I, d, INT64_MAX));
}

// Bands interleaved in the item order: at most 16, and near-equal groups (25 bands run as 13 + 12, not 16 + 9:
// a short last group would spread the CTAs over too many W tiles for L2).
int calib_tc_super_bands(int64_t bands)
{
    const int64_t groups = (bands + TC_SUPER_BANDS - 1) / TC_SUPER_BANDS;
    return (int)((bands + groups - 1) / groups);
}

int device_sm_count();   // dass_abi.cu

template <int ACT>
static cudaError_t launch_tc(const CUtensorMap &mx, const CUtensorMap &mg, const CUtensorMap &mu, const TcParams &p,
                             int grid, cudaStream_t st)
{
    static DeviceMask configured{0ull};               // per device
    const cudaError_t ce = ensure_dynamic_smem(calib_tc_kernel<ACT>, (int)TC_SMEM_BYTES, configured);
    if (ce != cudaSuccess) return ce;
    calib_tc_kernel<ACT><<<grid, TC_THREADS, TC_SMEM_BYTES, st>>>(mx, mg, mu, p);
    return cudaGetLastError();
}

// Self-test of the failure path: one thread waits, with the kernels' bounded wait, on an mbarrier that nothing will
// ever arrive at, and reports what the calibration kernels report when a wait runs out.
__global__ void bounded_wait_selftest_kernel(int *status, unsigned long long limit_ns)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const bool done = mbar_wait(smem_u32(&bar), 0u, &abort_flag, limit_ns);
        DASS_ST(status, done ? 0 : (int)DASS_ERR_TIMEOUT);
    }
}

cudaError_t bounded_wait_selftest_launch(int *status, unsigned long long limit_ns, cudaStream_t st)
{
    bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(status, limit_ns);
    return cudaGetLastError();
}

constexpr bool TC_USE_PAIR_KERNEL = true;   // layers with more than one neuron tile take the CTA-pair kernel (calib_tc2.cu)
dass_status calib_tc2_launch(const void *X, int64_t T, int64_t ldx, const void *Wg, const void *Wu,
                             int64_t I, int64_t d, int64_t ldw, int act, int band_tiles, double *partial, int *status,
                             cudaStream_t st);   // calib_tc2.cu

dass_status calib_tc_launch(const void *X, int64_t T, int64_t ldx, const void *Wg, const void *Wu,
                            int64_t I, int64_t d, int64_t ldw, int act, int band_tiles, double *partial, int *status,
                            cudaStream_t st)
{
    if (band_tiles < 1 || band_tiles > TC_MAX_BAND_TILES) return DASS_ERR_UNSUPPORTED;
    if (TC_USE_PAIR_KERNEL && I > TC_BM)
        return calib_tc2_launch(X, T, ldx, Wg, Wu, I, d, ldw, act, band_tiles, partial, status, st);
    if (d > 0x7fffffffll - TC_BK || T > 0x7fffffffll - TC_BN || I > 0x7fffffffll - TC_BM) return DASS_ERR_UNSUPPORTED;
    CUtensorMap mx, mg, mu;
    if (!tc_make_map(&mx, X, T, d, ldx, TC_BN) || !tc_make_map(&mg, Wg, I, d, ldw, TC_BM) || !tc_make_map(&mu, Wu, I, d, ldw, TC_BM))
        return DASS_ERR_CUDA;
    TcParams p;
    p.partial = partial; p.status = status; p.align_counter = status + 1;
    p.T = T; p.I = I; p.d = d;
    p.neuron_tiles = (I + TC_BM - 1) / TC_BM;
    p.token_tiles = (T + TC_BN - 1) / TC_BN;
    p.band_tiles = band_tiles;
    p.bands = calib_tc_parts_for(T, band_tiles);
    p.super_bands = calib_tc_super_bands(p.bands);
    p.items = p.neuron_tiles * p.bands;
    p.k_blocks = (d + TC_BK - 1) / TC_BK;
    const int sms = device_sm_count();
    const int grid = (int)(p.items < sms ? p.items : sms);
    cudaError_t e;
    switch (act) {
    case DASS_ACT_SILU: e = launch_tc<DASS_ACT_SILU>(mx, mg, mu, p, grid, st); break;
    case DASS_ACT_GELU_TANH: e = launch_tc<DASS_ACT_GELU_TANH>(mx, mg, mu, p, grid, st); break;
    default: e = launch_tc<DASS_ACT_RELU>(mx, mg, mu, p, grid, st); break;
    }
    return e == cudaSuccess ? DASS_OK : DASS_ERR_CUDA;
}

}  // namespace dass
