// Stage (a) for bf16 inputs, CTA-pair version: the same fused GLU GEMM as calib_tc.cu, but two CTAs (the two
// SMs of a TPC, a cluster of 2) drive one tcgen05.mma.cta_group::2 of shape 256 x 256:
//
//   * each CTA owns 128 neurons (its own Wg and Wu tiles, TMEM lanes 0..127 of its own SM) and loads only HALF of
//     the 256-token X tile; the hardware feeds both halves of B to both tensor cores.  Per k-slice a CTA therefore
//     moves 48 KB through shared memory instead of 64 KB and its MMAs read 64 KB instead of 96 KB -- the
//     single-CTA kernel is limited by exactly that shared-memory traffic (writes 64 + reads 96 bytes per clock
//     against 128 available).
//   * the leader CTA (cluster rank 0) issues all MMAs; both CTAs' TMA loads complete on the leader's "full"
//     barrier; tcgen05.commit multicasts the "slot free" and "accumulators ready" arrivals to both CTAs; the
//     peer's epilogue warps release the accumulators with remote mbarrier arrives.
//   * no TMA multicast is used anywhere.
//   * the accumulators G and U fill all 512 TMEM columns, so the next tile's MMAs cannot start before the epilogue has
//     READ them -- but they need not wait for its arithmetic.  Eight epilogue warps (two per TMEM lane quarter, each
//     taking half of the tile's 256 token columns) pull the accumulators into registers in chunks of 16 columns,
//     six chunks deep (the producer / MMA warpgroup gives its registers up with setmaxnreg so that the epilogue
//     warpgroups can hold them); after two chunks of arithmetic every column has been read and the accumulators are
//     handed back, the remaining six chunks are worked off out of registers under the next tile's MMAs.  The wait
//     the tensor cores see per tile falls from the whole epilogue (2 MUFU per element: about 4.1 k cycles) to about
//     a quarter of it.  The two warps of a lane quarter add their sums into the band's partial with one atomicAdd
//     each onto a zeroed slot: two addends, so the order does not matter and the result stays bit-reproducible.
// Everything else (item order, tile-boundary alignment barrier, L2 eviction hints, lane = neuron epilogue,
// per-band partial sums, bounded waits) is as in calib_tc.cu.
#include "tc_common.cuh"
#include "tc_pair.cuh"

namespace dass {

constexpr int T2_BM = 128;          // neurons per CTA (256 per pair)
constexpr int T2_BN = 256;          // tokens per tile (each CTA loads 128 of them)
constexpr int T2_BK = 64;
constexpr int T2_UMMA_K = 16;
constexpr int T2_STAGES = 4;
constexpr unsigned long long T2_ALIGN_NS = 20000ull;
constexpr int T2_EPI_WARPS = 8;      // two per TMEM lane quarter
constexpr int T2_CHUNK = 16;         // accumulator columns per register chunk
constexpr int T2_HELD = 6;           // chunks a thread holds at a time (g and u: 192 registers)
constexpr int T2_THREADS = 128 + 32 * T2_EPI_WARPS;   // warpgroup 0: TMA producer, MMA issuer, two idle warps; warpgroups 1, 2: epilogue
// Register split (setmaxnreg): 384 threads are launched with 168 registers each = 64512; 128 x 56 + 256 x 224 = 64512.
constexpr int T2_REGS_LAUNCH = 168, T2_REGS_CONTROL = 56, T2_REGS_EPILOGUE = 224;
static_assert(128 * T2_REGS_CONTROL + 32 * T2_EPI_WARPS * T2_REGS_EPILOGUE <= T2_THREADS * T2_REGS_LAUNCH, "setmaxnreg split exceeds the launch");
constexpr uint32_t T2_TILE_BYTES = 128 * T2_BK * 2;                 // 16 KB: a 128-row, 64-column bf16 tile
constexpr uint32_t T2_STAGE_BYTES = 3 * T2_TILE_BYTES;              // Wg + Wu + X half = 48 KB per CTA
constexpr uint32_t T2_TMEM_COLS = 512;
constexpr uint32_t T2_SMEM_BYTES = T2_STAGES * T2_STAGE_BYTES + 1024 + 256;

struct T2Params {
    double *partial;     // [bands][I]
    int *status;
    int *align_counter;
    int64_t T, I, d;
    int64_t neuron_pairs, token_tiles, bands, items, k_blocks;   // items = neuron_pairs * bands (one per CTA pair)
    int band_tiles;      // token tiles per band (calib_tc_band_tiles)
    int super_bands;     // bands interleaved in the item order (calib_tc_super_bands)
};

struct T2Item { int64_t np, band; };

__device__ __forceinline__ T2Item t2_decode(const T2Params &p, int64_t idx)
{
    const int64_t per_super = p.neuron_pairs * p.super_bands;
    const int64_t sb = idx / per_super;
    const int64_t rem = idx - sb * per_super;
    const int64_t left = p.bands - sb * p.super_bands;
    const int64_t nb = left < p.super_bands ? left : p.super_bands;
    T2Item c;
    c.np = rem / nb;
    c.band = sb * p.super_bands + (rem - c.np * nb);
    return c;
}

template <int ACT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(T2_THREADS, 1)
calib_tc2_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_wg,
                 const __grid_constant__ CUtensorMap map_wu, const T2Params p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *aligned = smem_raw + (base - raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(aligned + T2_STAGES * T2_STAGE_BYTES);
    const uint32_t bar_full = smem_u32(bars);                     // [T2_STAGES], used in the leader CTA only
    const uint32_t bar_empty = bar_full + 8 * T2_STAGES;          // [T2_STAGES], one set per CTA
    const uint32_t bar_acc_full = bar_empty + 8 * T2_STAGES;      // per CTA
    const uint32_t bar_acc_empty = bar_acc_full + 8;              // leader CTA only: both CTAs' epilogue warps arrive
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * T2_STAGES + 2);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                      // 0 = leader
    const int64_t cluster_id = blockIdx.x >> 1;
    const int64_t nclusters = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < T2_STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_acc_full, 1);
        mbar_init(bar_acc_empty, 2 * T2_EPI_WARPS);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(tmem_slot), T2_TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();            // both CTAs' barriers are initialised and both TMEM allocations exist
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(T2_REGS_CONTROL));
    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (one per CTA)
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            const uint64_t pol_w = l2_policy_evict_last();
            const uint64_t pol_x = l2_policy_evict_first();
            const uint32_t leader_full = map_to_cta(bar_full, 0);
            int64_t round = 0;
            for (int64_t idx = cluster_id; idx < p.items && ok; idx += nclusters, ++round) {
                const T2Item c = t2_decode(p, idx);
                const int64_t tt0 = c.band * p.band_tiles;
                const int64_t tt1 = tt0 + p.band_tiles < p.token_tiles ? tt0 + p.band_tiles : p.token_tiles;
                const int64_t left = p.items - round * nclusters;
                const int round_ctas = 2 * (int)(left < nclusters ? left : nclusters);
                const int w_row = (int)(c.np * 2 * T2_BM + rank * T2_BM);
                for (int64_t tt = tt0; tt < tt1 && ok; ++tt) {
                    {   // tile-boundary alignment of all CTAs of the round (bounded wait), see calib_tc.cu
                        const int t_in_item = (int)(tt - tt0);
                        const int target = (int)(round * gridDim.x) * p.band_tiles + round_ctas * (t_in_item + 1);
                        atomicAdd(p.align_counter, 1);
                        const unsigned long long t0 = global_ns();
                        while (*reinterpret_cast<volatile int *>(p.align_counter) < target && global_ns() - t0 < T2_ALIGN_NS) { }
                    }
                    const int x_row = (int)(tt * T2_BN + rank * (T2_BN / 2));
                    for (int64_t kb = 0; kb < p.k_blocks; ++kb) {
                        if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                        const uint32_t sbase = base + stage * T2_STAGE_BYTES;
                        const uint32_t fb = leader_full + 8 * stage;
                        if (rank == 0) mbar_arrive_expect_tx(bar_full + 8 * stage, 2 * T2_STAGE_BYTES);   // both CTAs' bytes
                        tma_load_2d_pair(sbase, &map_wg, fb, (int)(kb * T2_BK), w_row, pol_w);
                        tma_load_2d_pair(sbase + T2_TILE_BYTES, &map_wu, fb, (int)(kb * T2_BK), w_row, pol_w);
                        tma_load_2d_pair(sbase + 2 * T2_TILE_BYTES, &map_x, fb, (int)(kb * T2_BK), x_row, pol_x);
                        if (++stage == T2_STAGES) { stage = 0; phase ^= 1u; }
                    }
                }
                if (tt1 - tt0 < p.band_tiles) atomicAdd(p.align_counter, (int)(p.band_tiles - (tt1 - tt0)));
            }
            if (!ok) { *abort_flag = 1; atomicExch(p.status, (int)DASS_ERR_TIMEOUT); }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = idesc_bf16_f32(2 * T2_BM, T2_BN);
            uint32_t stage = 0, phase = 0, tile = 0;
            bool ok = true;
            for (int64_t idx = cluster_id; idx < p.items && ok; idx += nclusters) {
                const T2Item c = t2_decode(p, idx);
                const int64_t tt0 = c.band * p.band_tiles;
                const int64_t tt1 = tt0 + p.band_tiles < p.token_tiles ? tt0 + p.band_tiles : p.token_tiles;
                for (int64_t tt = tt0; tt < tt1 && ok; ++tt, ++tile) {
                    if (!mbar_wait(bar_acc_empty, (tile & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    for (int64_t kb = 0; kb < p.k_blocks; ++kb) {
                        if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t sbase = base + stage * T2_STAGE_BYTES;
                        const uint64_t dg = smem_desc_sw128(sbase);
                        const uint64_t du = smem_desc_sw128(sbase + T2_TILE_BYTES);
                        const uint64_t dx = smem_desc_sw128(sbase + 2 * T2_TILE_BYTES);
#pragma unroll
                        for (int k = 0; k < T2_BK / T2_UMMA_K; ++k) {
                            const uint32_t acc = (kb > 0 || k > 0) ? 1u : 0u;
                            const uint64_t koff = (uint64_t)(k * T2_UMMA_K * 2 / 16);
                            umma_bf16_pair(tmem_base, dg + koff, dx + koff, idesc, acc);
                            umma_bf16_pair(tmem_base + T2_BN, du + koff, dx + koff, idesc, acc);
                        }
                        umma_commit_pair(bar_empty + 8 * stage, (uint16_t)3);   // slot free in both CTAs
                        if (++stage == T2_STAGES) { stage = 0; phase ^= 1u; }
                    }
                    if (ok) umma_commit_pair(bar_acc_full, (uint16_t)3);        // accumulators ready in both CTAs
                }
            }
            if (!ok) { *abort_flag = 1; atomicExch(p.status, (int)DASS_ERR_TIMEOUT); }
        }
        __syncwarp();
    }
    } else {
        // ------------------------------------------------------------ epilogue (8 warps, this CTA's 128 neurons)
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(T2_REGS_EPILOGUE));
        constexpr int NCHUNK = (T2_BN / 2) / T2_CHUNK;        // chunks per warp: its half of the tile's token columns
        static_assert(NCHUNK > T2_HELD && NCHUNK - T2_HELD < T2_HELD, "refills reuse the chunks computed first");
        const int quad = warp & 3;                            // the TMEM lane quarter this warp may read
        const int half = (warp - 4) >> 2;                     // which 128 of the 256 token columns
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(half * (T2_BN / 2));
        const uint32_t leader_acc_empty = map_to_cta(bar_acc_empty, 0);
        uint32_t tile = 0;
        bool ok = true;
        for (int64_t idx = cluster_id; idx < p.items && ok; idx += nclusters) {
            const T2Item c = t2_decode(p, idx);
            const int64_t tt0 = c.band * p.band_tiles;
            const int64_t tt1 = tt0 + p.band_tiles < p.token_tiles ? tt0 + p.band_tiles : p.token_tiles;
            double acc = 0.0;
            for (int64_t tt = tt0; tt < tt1 && ok; ++tt, ++tile) {
                if (!mbar_wait(bar_acc_full, tile & 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                float s = 0.0f;
                uint32_t g[T2_HELD][T2_CHUNK], u[T2_HELD][T2_CHUNK];
#pragma unroll
                for (int ch = 0; ch < T2_HELD; ++ch) {
                    tmem_ld_16(lane_addr + ch * T2_CHUNK, g[ch]);
                    tmem_ld_16(lane_addr + T2_BN + ch * T2_CHUNK, u[ch]);
                }
                tmem_wait_ld();
#pragma unroll
                for (int ch = 0; ch < NCHUNK; ++ch) {
                    const int b = ch % T2_HELD;
#pragma unroll
                    for (int j = 0; j < T2_CHUNK; ++j) {
                        const float h = glu_h<ACT>(__uint_as_float(g[b][j]), __uint_as_float(u[b][j]));
                        s = fmaf(h, h, s);
                    }
                    if (ch + T2_HELD < NCHUNK) {              // the registers just used take a chunk not read yet
                        tmem_ld_16(lane_addr + (ch + T2_HELD) * T2_CHUNK, g[b]);
                        tmem_ld_16(lane_addr + T2_BN + (ch + T2_HELD) * T2_CHUNK, u[b]);
                    }
                    if (ch + T2_HELD == NCHUNK - 1) {         // that was the last read: hand the accumulators back
                        tmem_wait_ld();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) {
                            if (rank == 0) mbar_arrive(bar_acc_empty);
                            else mbar_arrive_cluster(leader_acc_empty);
                        }
                    }
                }
                acc += (double)s;
            }
            const int64_t neuron = c.np * 2 * T2_BM + rank * T2_BM + quad * 32 + lane;
            if (ok && neuron < p.I && DASS_ACCESS_OK(&p.partial[c.band * p.I + neuron], 8))
                atomicAdd(&p.partial[c.band * p.I + neuron], acc);   // two addends onto a zeroed slot
        }
        if (!ok && lane == 0) { *abort_flag = 1; atomicExch(p.status, (int)DASS_ERR_TIMEOUT); }
    }
    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 20; ++i) __nanosleep(1000000);   // failure path: let issued copies / MMAs land
        __syncthreads();
    }
    cluster_sync_all();            // the peer no longer signals into this CTA's shared memory or uses the pair's TMEM
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, T2_TMEM_COLS);
    }
}

// ------------------------------------------------------------------ host side
bool tc_make_map(CUtensorMap *map, const void *ptr, int64_t rows, int64_t cols, int64_t ld, int box_rows);   // calib_tc.cu
int64_t calib_tc_parts_for(int64_t T, int band_tiles);                                                        // calib_tc.cu
int calib_tc_super_bands(int64_t bands);                                                                      // calib_tc.cu
int device_sm_count();                                                                                        // dass_abi.cu

template <int ACT>
static cudaError_t launch_tc2(const CUtensorMap &mx, const CUtensorMap &mg, const CUtensorMap &mu, const T2Params &p,
                              int grid, cudaStream_t st)
{
    static DeviceMask configured{0ull};               // per device
    const cudaError_t ce = ensure_dynamic_smem(calib_tc2_kernel<ACT>, (int)T2_SMEM_BYTES, configured);
    if (ce != cudaSuccess) return ce;
    calib_tc2_kernel<ACT><<<grid, T2_THREADS, T2_SMEM_BYTES, st>>>(mx, mg, mu, p);
    return cudaGetLastError();
}

// CTA-pair launch; same contract as calib_tc_launch (partials per band, status word, alignment counter behind it).
dass_status calib_tc2_launch(const void *X, int64_t T, int64_t ldx, const void *Wg, const void *Wu,
                             int64_t I, int64_t d, int64_t ldw, int act, int band_tiles, double *partial, int *status,
                             cudaStream_t st)
{
    if (d > 0x7fffffffll - T2_BK || T > 0x7fffffffll - T2_BN || I > 0x7fffffffll - 2 * T2_BM) return DASS_ERR_UNSUPPORTED;
    CUtensorMap mx, mg, mu;
    if (!tc_make_map(&mx, X, T, d, ldx, T2_BN / 2) || !tc_make_map(&mg, Wg, I, d, ldw, T2_BM) ||
        !tc_make_map(&mu, Wu, I, d, ldw, T2_BM))
        return DASS_ERR_CUDA;
    T2Params p;
    p.partial = partial; p.status = status; p.align_counter = status + 1;
    p.T = T; p.I = I; p.d = d;
    p.neuron_pairs = (I + 2 * T2_BM - 1) / (2 * T2_BM);
    p.token_tiles = (T + T2_BN - 1) / T2_BN;
    p.band_tiles = band_tiles;
    p.bands = calib_tc_parts_for(T, band_tiles);
    p.super_bands = calib_tc_super_bands(p.bands);
    p.items = p.neuron_pairs * p.bands;
    p.k_blocks = (d + T2_BK - 1) / T2_BK;
    const int64_t max_pairs = device_sm_count() / 2;
    const int grid = 2 * (int)(p.items < max_pairs ? p.items : max_pairs);
    // the two epilogue warps of a lane quarter add into the partials: they start from zero
    if (cudaMemsetAsync(partial, 0, (size_t)p.bands * (size_t)I * sizeof(double), st) != cudaSuccess) return DASS_ERR_CUDA;
    cudaError_t e;
    switch (act) {
    case DASS_ACT_SILU: e = launch_tc2<DASS_ACT_SILU>(mx, mg, mu, p, grid, st); break;
    case DASS_ACT_GELU_TANH: e = launch_tc2<DASS_ACT_GELU_TANH>(mx, mg, mu, p, grid, st); break;
    default: e = launch_tc2<DASS_ACT_RELU>(mx, mg, mu, p, grid, st); break;
    }
    return e == cudaSuccess ? DASS_OK : DASS_ERR_CUDA;
}

}  // namespace dass
