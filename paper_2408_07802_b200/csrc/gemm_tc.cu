// Grouped bf16 GEMM  C_g[M, Nout] = A_g[M, K] . W_g[Nout, K]^T  on the sm_100a tensor cores.
//
// One persistent CTA per SM, six warps:
//   warp 0    TMA producer: 128 x 64 tile of A and BN x 64 tile of W per stage, 128-byte swizzle;
//   warp 1    allocates TMEM and issues tcgen05.mma (128 x BN x 16 per instruction, fp32
//             accumulators in TMEM, two accumulator buffers so that draining tile i overlaps
//             the MMAs of tile i+1);
//   warps 2-9 epilogue: tcgen05.ld of their 32-lane quarter (two warps per quarter, each one half
//             of the tile's columns), fused epilogue, global stores.
// The group (branch) index is the outermost TMA coordinate.  Rows past M, columns past Nout
// and the K tail are zero-filled by TMA and masked in the epilogue.
//
// Tile order: the group is the slowest index, so the operands of one group (tens of MB) stay
// in L2 while its tiles are walked.  The down-projection's cross-branch sum (the AllReduce of
// Algorithm 1) instead needs the N groups of one output tile on the same CTA in ascending order
// (`group_serial`); there the dimension with fewer tiles runs fastest so that one wave of CTAs
// spans it completely and shares those operand tiles through L2.
#include <stdio.h>
#include <stdlib.h>

#include "epilogue.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace kr {

namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int EPI_WARPS = 8;
constexpr int NUM_THREADS = 64 + 32 * EPI_WARPS;
constexpr int SMEM_BUDGET = 200 * 1024;

template <int BN>
struct TileCfg {
    static constexpr int A_BYTES = BM * BK * 2;
    static constexpr int B_BYTES = BN * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = SMEM_BUDGET / STAGE_BYTES > 8 ? 8 : SMEM_BUDGET / STAGE_BYTES;
    // two accumulators; TMEM is allocated in powers of two of at least 32 columns
    static constexpr int TMEM_COLS = 2 * BN <= 64 ? 64 : (2 * BN <= 128 ? 128 : (2 * BN <= 256 ? 256 : 512));
    static constexpr int EPI_BIAS_BYTES = EPI_WARPS * 256;   // the epilogue warps' strips of bias values
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/ + EPI_BIAS_BYTES;
};

// 32-row slabs of one group as the fused LayerNorm counts them: every tile row, also past M, has its counters
__host__ __device__ constexpr int ln_slabs(int m) { return (m + 2 * BM - 1) / (2 * BM) * (2 * BM / 32); }

struct KernelArgs {
    GemmShape shape;
    EpiParams epi;
    int tiles_m, tiles_n;
    int a_gmul, b_gmul;  // 0 when the operand is shared by all groups
    int a_g0, b_g0;      // first group's index along the outermost TMA dimension
    int group_serial;
    int n_fastest;  // tile order inside a group: 1 = n-tiles fastest, 0 = m-tiles fastest
    int w_early;    // W is not the stream's previous kernel's to write: its first tiles are fetched before that one ends
    uint32_t *status;
};

__device__ __forceinline__ bool next_item(const KernelArgs &ka, int it, int &m_blk, int &n_blk, int &g) {
    const int G = ka.shape.groups;
    const int num_tiles = ka.tiles_m * ka.tiles_n;
    int tile;
    if (ka.group_serial) {
        tile = blockIdx.x + (it / G) * gridDim.x;
        g = it % G;
    } else {
        const long long idx = blockIdx.x + (long long)it * gridDim.x;
        g = static_cast<int>(idx / num_tiles);
        if (g >= G) return false;
        tile = static_cast<int>(idx % num_tiles);
    }
    if (tile >= num_tiles) return false;
    if (ka.n_fastest) {
        n_blk = tile % ka.tiles_n;
        m_blk = tile / ka.tiles_n;
    } else {
        m_blk = tile % ka.tiles_m;
        n_blk = tile / ka.tiles_m;
    }
    return true;
}

// LN: with a LayerNorm behind the epilogue.  A kernel of its own, so that the plain one carries none of its code.
template <int BN, bool LN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const KernelArgs ka) {
    using Cfg = TileCfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *tiles = smem;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + Cfg::STAGES * Cfg::STAGE_BYTES);
    uint64_t *full_bar = bars;                      // [STAGES]
    uint64_t *empty_bar = bars + Cfg::STAGES;       // [STAGES]
    uint64_t *acc_full = bars + 2 * Cfg::STAGES;    // [2]
    uint64_t *acc_empty = bars + 2 * Cfg::STAGES + 2;  // [2]
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * Cfg::STAGES + 4);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k_blocks = (ka.shape.k + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < Cfg::STAGES; ++s) {
            mbar_init(full_bar + s, 1);
            mbar_init(empty_bar + s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(acc_full + a, 1);
            mbar_init(acc_empty + a, EPI_WARPS);
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Launched ahead of the end of its predecessor: nothing of the predecessor's is touched before pdl_wait().  The
    // weights are not the predecessor's, so the W tiles of the first stages are on their way while it drains.
    int pre = 0;
    if (threadIdx.x == 0 && ka.w_early) {
        int m_blk, n_blk, g;
        if (next_item(ka, 0, m_blk, n_blk, g)) {
            pre = k_blocks < Cfg::STAGES ? k_blocks : Cfg::STAGES;
            for (int kb = 0; kb < pre; ++kb) {
                mbar_expect_tx(full_bar + kb, Cfg::STAGE_BYTES);
                tma_load_3d(tiles + kb * Cfg::STAGE_BYTES + Cfg::A_BYTES, &tmB, full_bar + kb, kb * BK, n_blk * BN,
                            ka.b_g0 + g * ka.b_gmul);
            }
        }
    }
    pdl_wait();
    pdl_trigger();   // the successor's CTAs may take this one's place as soon as it leaves

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int m_blk, n_blk, g;
            for (int it = 0; ok && next_item(ka, it, m_blk, n_blk, g); ++it) {
                for (int kb = 0; kb < k_blocks; ++kb) {
                    const bool early = it == 0 && kb < pre;   // stage kb, armed, its W tile under way
                    if (!early && !(ok = mbar_wait(empty_bar + stage, phase ^ 1u, abort_flag))) break;
                    uint8_t *sa = tiles + stage * Cfg::STAGE_BYTES;
                    uint8_t *sb = sa + Cfg::A_BYTES;
                    if (!early) mbar_expect_tx(full_bar + stage, Cfg::STAGE_BYTES);
                    tma_load_3d(sa, &tmA, full_bar + stage, kb * BK, m_blk * BM, ka.a_g0 + g * ka.a_gmul);
                    if (!early) tma_load_3d(sb, &tmB, full_bar + stage, kb * BK, n_blk * BN, ka.b_g0 + g * ka.b_gmul);
                    if (++stage == Cfg::STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_h16(BM, BN);
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            int m_blk, n_blk, g;
            for (int it = 0; ok && next_item(ka, it, m_blk, n_blk, g); ++it) {
                if (!(ok = mbar_wait(acc_empty + acc, acc_phase ^ 1u, abort_flag))) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!(ok = mbar_wait(full_bar + stage, phase, abort_flag))) break;
                    tc_fence_after_sync();
                    const uint32_t sa = smem_u32(tiles + stage * Cfg::STAGE_BYTES);
                    const uint32_t sb = sa + Cfg::A_BYTES;
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        umma_bf16_ss(d_tmem, umma_desc_sw128_kmajor(sa + k * UMMA_K * 2),
                                     umma_desc_sw128_kmajor(sb + k * UMMA_K * 2), idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    umma_commit(empty_bar + stage);  // frees the stage once these MMAs have read it
                    if (++stage == Cfg::STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                umma_commit(acc_full + acc);  // accumulator complete
                if (++acc == 2) {
                    acc = 0;
                    acc_phase ^= 1u;
                }
            }
        }
        __syncwarp();
    } else {
        const int quarter = warp & 3;          // TMEM lanes this warp may read
        const int half = (warp - 2) >> 2;      // which half of the tile's columns it drains
        constexpr int CHUNKS = BN / 32;        // 32-column chunks of the tile: `half` takes every second one
        constexpr bool ln = LN;
        uint16_t *bias_strip = reinterpret_cast<uint16_t *>(smem + Cfg::STAGES * Cfg::STAGE_BYTES + 256) + (warp - 2) * 128;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        int m_blk, n_blk, g;
        for (int it = 0; ok && next_item(ka, it, m_blk, n_blk, g); ++it) {
            // the bias of this warp's chunks (chunk half + 2 i at values 32 i .. 32 i + 31), fetched while the MMAs run
            if (!ln && ka.epi.bias)
                park_bias(ka.epi.bias + g * ka.epi.bias_gstride,
                          n_blk * BN + (half + 2 * (lane >> 3)) * 32 + 4 * (lane & 7), ka.shape.n_out, bias_strip, lane);
            ok = mbar_wait(acc_full + acc, acc_phase, abort_flag);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const int row = m_blk * BM + quarter * 32 + lane;
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                                   static_cast<uint32_t>(acc * BN);
            if (!ln) {
#pragma unroll 1
                for (int c = half; c < CHUNKS; c += 2) {
                    const int col0 = n_blk * BN + c * 32;
                    if (col0 >= ka.shape.n_out) break;  // uniform across the warp
                    uint32_t r[32];
                    tmem_ld_32x32(t_row + static_cast<uint32_t>(c * 32), r);
                    tmem_ld_wait();
                    if (row < ka.shape.m) {
                        float v[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
                        const int ncols = min(32, ka.shape.n_out - col0);
                        if (ka.epi.bias) add_bias_chunk_parked(bias_strip + (c >> 1) * 32, v);   // (zeros past n_out)
                        epilogue_chunk(ka.epi, g, row, col0, ncols, v, false);
                    }
                }
            }
            RowStats rs{0.f, 0.f, 0.f};
            if (ln) {
                // first pass with a LayerNorm behind it: the same epilogue, the row statistics, and the row the
                // LayerNorm sees back into the accumulator's columns
#pragma unroll 1
                for (int c = half; c < CHUNKS; c += 2) {
                    const int col0 = n_blk * BN + c * 32;
                    if (col0 >= ka.shape.n_out) break;
                    uint32_t r[32];
                    tmem_ld_32x32(t_row + static_cast<uint32_t>(c * 32), r);
                    tmem_ld_wait();
                    const int ncols = min(32, ka.shape.n_out - col0);
                    if (row < ka.shape.m) {
                        float v[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
                        epilogue_chunk_ln(ka.epi, g, row, col0, ncols, v);
                        stats_add_chunk(rs, v, ncols);
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(v[i]);
                    }
                    tmem_st_32x32(t_row + static_cast<uint32_t>(c * 32), r);
                }
            }
            if (ln) {
                // the row's other columns are other CTAs' tiles: leave this part's statistics, wait for the rest
                tmem_st_wait();
                const int n_parts = ka.epi.ln_n_parts;
                float4 *parts = ka.epi.ln_parts + ((long long)g * ka.shape.m + row) * n_parts;
                if (row < ka.shape.m) parts[n_blk * 2 + half] = make_float4(rs.mean, rs.m2, rs.cnt, 0.f);
                uint32_t *cnt = ka.epi.ln_cnt + ((long long)g * ln_slabs(ka.shape.m) + m_blk * (BM / 32) + quarter) * 2;
                ok = ln_arrive_and_wait(cnt, n_parts, lane, abort_flag);
                if (!ok) break;
                float mean = 0.f, rstd = 0.f;
                if (row < ka.shape.m) ln_row_stats(parts, n_parts, ka.epi.ln_eps, mean, rstd);
#pragma unroll 1
                for (int c = half; c < CHUNKS; c += 2) {
                    const int col0 = n_blk * BN + c * 32;
                    if (col0 >= ka.shape.n_out) break;
                    uint32_t r[32];
                    tmem_ld_32x32(t_row + static_cast<uint32_t>(c * 32), r);
                    tmem_ld_wait();
                    if (row < ka.shape.m) {
                        float z[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) z[i] = __uint_as_float(r[i]);
                        ln_store_chunk(ka.epi, g, row, col0, min(32, ka.shape.n_out - col0), z, mean, rstd);
                    }
                }
                ln_depart(cnt, n_parts, lane);
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty + acc);
            if (++acc == 2) {
                acc = 0;
                acc_phase ^= 1u;
            }
        }
    }

    // teardown (also reached when a bounded wait gave up)
    if (*abort_flag) {
        // give copies and MMAs still in flight time to land before shared memory and TMEM go away
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
        if (threadIdx.x == 0 && ka.status) atomicOr(ka.status, STATUS_WAIT_LIMIT);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
}

// ------------------------------------------------------------------------------------------------
// CTA-pair version: two CTAs of a cluster work on one 256 x 256 output tile.  Each CTA loads its 128
// rows of A and HALF of the W tile (128 rows), the leader issues tcgen05.mma.cta_group::2 (256 x 256
// x 16), and each CTA's tensor core reads both halves of W, so every W byte is fetched into shared
// memory once per pair instead of once per CTA: a third less shared-memory traffic per flop, which
// is what bounds the single-CTA 128 x 256 tile.  Each CTA drains its own 128 accumulator rows.
// Barriers: `full` lives in the leader (both CTAs' TMA loads report their bytes to it), `empty` and
// `acc_full` exist in both CTAs and are signalled by multicast commits, `acc_empty` lives in the
// leader and collects the epilogue warps of both CTAs.
// ------------------------------------------------------------------------------------------------

constexpr int BN2 = 256;

struct PairCfg {
    static constexpr int A_BYTES = BM * BK * 2;            // 128 rows of A
    static constexpr int B_BYTES = (BN2 / 2) * BK * 2;     // this CTA's half of the W tile
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = 5;
    static constexpr int TMEM_COLS = 2 * BN2;
    static constexpr int EPI_STAGE_BYTES = EPI_WARPS * EPI_STAGE_FLOATS * 4;  // fp32 epilogue staging tiles
    static constexpr int EPI_BIAS_BYTES = EPI_WARPS * 256;   // and their strips of bias values (128 columns each)
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 256 + EPI_STAGE_BYTES + EPI_BIAS_BYTES;
};

__device__ __forceinline__ bool next_item_pair(const KernelArgs &ka, int it, int cluster_id, int n_clusters,
                                               int &m_blk, int &n_blk, int &g) {
    const int G = ka.shape.groups;
    const int tiles_m = (ka.shape.m + 2 * BM - 1) / (2 * BM);
    const int num_tiles = tiles_m * ka.tiles_n;
    int tile;
    if (ka.group_serial) {
        tile = cluster_id + (it / G) * n_clusters;
        g = it % G;
    } else {
        const long long idx = cluster_id + (long long)it * n_clusters;
        g = static_cast<int>(idx / num_tiles);
        if (g >= G) return false;
        tile = static_cast<int>(idx % num_tiles);
    }
    if (tile >= num_tiles) return false;
    if (ka.n_fastest) {
        n_blk = tile % ka.tiles_n;
        m_blk = tile / ka.tiles_n;
    } else {
        m_blk = tile % tiles_m;
        n_blk = tile / tiles_m;
    }
    return true;
}

template <bool LN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const KernelArgs ka) {
    using Cfg = PairCfg;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *tiles = smem;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + Cfg::STAGES * Cfg::STAGE_BYTES);
    uint64_t *full_bar = bars;                         // [STAGES]  used in the leader
    uint64_t *empty_bar = bars + Cfg::STAGES;          // [STAGES]  both CTAs
    uint64_t *acc_full = bars + 2 * Cfg::STAGES;       // [2]       both CTAs
    uint64_t *acc_empty = bars + 2 * Cfg::STAGES + 2;  // [2]       used in the leader
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * Cfg::STAGES + 4);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
    const int k_blocks = (ka.shape.k + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < Cfg::STAGES; ++s) {
            mbar_init(full_bar + s, 1);
            mbar_init(empty_bar + s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(acc_full + a, 1);
            mbar_init(acc_empty + a, 2 * EPI_WARPS);
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, Cfg::TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();  // both CTAs' barriers exist before anything is signalled across the pair
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // (see the single-CTA kernel: the first stages' W tiles are fetched while the predecessor drains)
    int pre = 0;
    if (threadIdx.x == 0 && ka.w_early) {
        int m_blk, n_blk, g;
        if (next_item_pair(ka, 0, cluster_id, n_clusters, m_blk, n_blk, g)) {
            pre = k_blocks < Cfg::STAGES ? k_blocks : Cfg::STAGES;
            for (int kb = 0; kb < pre; ++kb) {
                if (rank == 0) mbar_expect_tx(full_bar + kb, 2 * Cfg::STAGE_BYTES);
                tma_load_3d_pair(tiles + kb * Cfg::STAGE_BYTES + Cfg::A_BYTES, &tmB, map_to_cta(smem_u32(full_bar + kb), 0),
                                 kb * BK, n_blk * BN2 + (int)rank * (BN2 / 2), ka.b_g0 + g * ka.b_gmul);
            }
        }
    }
    pdl_wait();
    pdl_trigger();

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int m_blk, n_blk, g;
            for (int it = 0; ok && next_item_pair(ka, it, cluster_id, n_clusters, m_blk, n_blk, g); ++it) {
                for (int kb = 0; kb < k_blocks; ++kb) {
                    const bool early = it == 0 && kb < pre;
                    if (!early && !(ok = mbar_wait(empty_bar + stage, phase ^ 1u, abort_flag))) break;
                    uint8_t *sa = tiles + stage * Cfg::STAGE_BYTES;
                    uint8_t *sb = sa + Cfg::A_BYTES;
                    const uint32_t leader_full = map_to_cta(smem_u32(full_bar + stage), 0);
                    if (rank == 0 && !early) mbar_expect_tx(full_bar + stage, 2 * Cfg::STAGE_BYTES);
                    tma_load_3d_pair(sa, &tmA, leader_full, kb * BK, m_blk * 2 * BM + (int)rank * BM,
                                     ka.a_g0 + g * ka.a_gmul);
                    if (!early)
                        tma_load_3d_pair(sb, &tmB, leader_full, kb * BK, n_blk * BN2 + (int)rank * (BN2 / 2),
                                         ka.b_g0 + g * ka.b_gmul);
                    if (++stage == Cfg::STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = umma_idesc_h16(2 * BM, BN2);
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            int m_blk, n_blk, g;
            for (int it = 0; ok && next_item_pair(ka, it, cluster_id, n_clusters, m_blk, n_blk, g); ++it) {
                if (!(ok = mbar_wait(acc_empty + acc, acc_phase ^ 1u, abort_flag))) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN2);
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!(ok = mbar_wait(full_bar + stage, phase, abort_flag))) break;
                    tc_fence_after_sync();
                    const uint32_t sa = smem_u32(tiles + stage * Cfg::STAGE_BYTES);
                    const uint32_t sb = sa + Cfg::A_BYTES;
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        umma_bf16_ss_pair(d_tmem, umma_desc_sw128_kmajor(sa + k * UMMA_K * 2),
                                          umma_desc_sw128_kmajor(sb + k * UMMA_K * 2), idesc,
                                          (kb | k) != 0 ? 1u : 0u);
                    }
                    umma_commit_pair(empty_bar + stage, 3);  // frees the stage in both CTAs
                    if (++stage == Cfg::STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                umma_commit_pair(acc_full + acc, 3);  // accumulator complete in both CTAs
                if (++acc == 2) {
                    acc = 0;
                    acc_phase ^= 1u;
                }
            }
        }
        __syncwarp();
    } else {
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;
        constexpr int CHUNKS = BN2 / 32 / 2;
        float *stage = reinterpret_cast<float *>(smem + Cfg::STAGES * Cfg::STAGE_BYTES + 256) +
                       (warp - 2) * EPI_STAGE_FLOATS;
        uint16_t *bias_strip = reinterpret_cast<uint16_t *>(smem + Cfg::STAGES * Cfg::STAGE_BYTES + 256 +
                                                            Cfg::EPI_STAGE_BYTES) + (warp - 2) * 128;
        const bool staged = epilogue_f32_stageable(ka.epi);
        constexpr bool ln = LN;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        int m_blk, n_blk, g;
        for (int it = 0; ok && next_item_pair(ka, it, cluster_id, n_clusters, m_blk, n_blk, g); ++it) {
            // the bias of this warp's 128 columns, fetched while the MMAs of the tile run
            if (ka.epi.bias)
                park_bias(ka.epi.bias + g * ka.epi.bias_gstride, n_blk * BN2 + half * (BN2 / 2) + 4 * lane, ka.shape.n_out,
                          bias_strip, lane);
            const int row_base = m_blk * 2 * BM + (int)rank * BM + quarter * 32;
            const int row = row_base + lane;
            ok = mbar_wait(acc_full + acc, acc_phase, abort_flag);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                                   static_cast<uint32_t>(acc * BN2);
            if (!ln) {
#pragma unroll 1
                for (int cc = 0; cc < CHUNKS; ++cc) {
                    const int c = half * CHUNKS + cc;
                    const int col0 = n_blk * BN2 + c * 32;
                    if (col0 >= ka.shape.n_out) break;
                    uint32_t r[32];
                    tmem_ld_32x32(t_row + static_cast<uint32_t>(c * 32), r);
                    tmem_ld_wait();
                    if (staged && col0 + 32 <= ka.shape.n_out) {
                        // coalesced path: the whole warp takes part, rows past M are masked inside
                        float v[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
                        if (ka.epi.bias) add_bias_chunk_parked(bias_strip + cc * 32, v);
                        epilogue_f32_staged(ka.epi, g, row_base, ka.shape.m, col0, v, stage, lane);
                    } else if (row < ka.shape.m) {
                        float v[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
                        const int ncols = min(32, ka.shape.n_out - col0);
                        if (ka.epi.bias) add_bias_chunk_parked(bias_strip + cc * 32, v);   // (zeros past n_out)
                        epilogue_chunk(ka.epi, g, row, col0, ncols, v, false);
                    }
                }
            }
            RowStats rs{0.f, 0.f, 0.f};
            if (ln) {
                // first pass with a LayerNorm behind it (see the single-CTA kernel)
#pragma unroll 1
                for (int cc = 0; cc < CHUNKS; ++cc) {
                    const int c = half * CHUNKS + cc;
                    const int col0 = n_blk * BN2 + c * 32;
                    if (col0 >= ka.shape.n_out) break;
                    uint32_t r[32];
                    tmem_ld_32x32(t_row + static_cast<uint32_t>(c * 32), r);
                    tmem_ld_wait();
                    const int ncols = min(32, ka.shape.n_out - col0);
                    if (staged && col0 + 32 <= ka.shape.n_out) {
                        float v[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
                        if (ka.epi.bias) add_bias_chunk(ka.epi.bias + g * ka.epi.bias_gstride + col0, v, 32);
                        epilogue_f32_staged(ka.epi, g, row_base, ka.shape.m, col0, v, stage, lane, true);
                        if (row < ka.shape.m) stats_add_chunk(rs, v, 32);
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(v[i]);
                    } else if (row < ka.shape.m) {
                        float v[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
                        epilogue_chunk_ln(ka.epi, g, row, col0, ncols, v);
                        stats_add_chunk(rs, v, ncols);
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(v[i]);
                    }
                    tmem_st_32x32(t_row + static_cast<uint32_t>(c * 32), r);
                }
            }
            if (ln) {
                tmem_st_wait();
                const int n_parts = ka.epi.ln_n_parts;
                float4 *parts = ka.epi.ln_parts + ((long long)g * ka.shape.m + row) * n_parts;
                if (row < ka.shape.m) parts[n_blk * 2 + half] = make_float4(rs.mean, rs.m2, rs.cnt, 0.f);
                uint32_t *cnt = ka.epi.ln_cnt + ((long long)g * ln_slabs(ka.shape.m) + row_base / 32) * 2;
                ok = ln_arrive_and_wait(cnt, n_parts, lane, abort_flag);
                if (!ok) break;
                float mean = 0.f, rstd = 0.f;
                if (row < ka.shape.m) ln_row_stats(parts, n_parts, ka.epi.ln_eps, mean, rstd);
#pragma unroll 1
                for (int cc = 0; cc < CHUNKS; ++cc) {
                    const int c = half * CHUNKS + cc;
                    const int col0 = n_blk * BN2 + c * 32;
                    if (col0 >= ka.shape.n_out) break;
                    uint32_t r[32];
                    tmem_ld_32x32(t_row + static_cast<uint32_t>(c * 32), r);
                    tmem_ld_wait();
                    if (row < ka.shape.m) {
                        float z[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) z[i] = __uint_as_float(r[i]);
                        ln_store_chunk(ka.epi, g, row, col0, min(32, ka.shape.n_out - col0), z, mean, rstd);
                    }
                }
                ln_depart(cnt, n_parts, lane);
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(acc_empty + acc), 0));
            if (++acc == 2) {
                acc = 0;
                acc_phase ^= 1u;
            }
        }
    }

    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
        if (threadIdx.x == 0 && ka.status) atomicOr(ka.status, STATUS_WAIT_LIMIT);
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();  // nothing of the pair (remote arrivals, MMA reads of peer memory) is in flight
    if (warp == 1) tmem_dealloc_pair(tmem_base, Cfg::TMEM_COLS);
}

template <bool LN>
int launch_pair(const CUtensorMap &tmA, const CUtensorMap &tmB, const KernelArgs &ka, cudaStream_t stream) {
    using Cfg = PairCfg;
    static DeviceOnce configured;
    static std::atomic<int> max_clusters_of[MAX_DEVICES];
    const int dev = device_slot();
    if (dev < 0) return KRAKEN_ECUDA;
    if (!configured.done()) {
        int rc = cuda_check(cudaFuncSetAttribute(gemm_tc_pair_kernel<LN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 Cfg::SMEM_BYTES), "gemm pair: shared memory opt-in");
        if (rc) return rc;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * 148);
        cfg.blockDim = dim3(NUM_THREADS);
        cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2;
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, gemm_tc_pair_kernel<LN>, &cfg) != cudaSuccess || n < 1) {
            cudaGetLastError();
            n = (sm_count() > 0 ? sm_count() : 148) / 2;
        }
        max_clusters_of[dev].store(n);
        configured.set();
    }
    const int max_clusters = max_clusters_of[dev].load();
    const long long tiles = (long long)((ka.shape.m + 2 * BM - 1) / (2 * BM)) * ka.tiles_n;
    const long long units = ka.group_serial ? tiles : tiles * ka.shape.groups;
    int clusters = static_cast<int>(units < max_clusters ? units : max_clusters);
    // LayerNorm behind the epilogue: the N tiles of a row block wait for each other, so a round of clusters must
    // hold whole row blocks (a block split over two rounds stalls its first part for a whole tile, every round)
    if (ka.epi.ln_out && clusters > ka.tiles_n) clusters -= clusters % ka.tiles_n;
    return cuda_check(launch_pdl(gemm_tc_pair_kernel<LN>, dim3(2 * clusters), dim3(NUM_THREADS), Cfg::SMEM_BYTES, stream, tmA, tmB, ka),
                      "gemm pair: launch");
}

template <int BN, bool LN>
int launch_bn_as(const CUtensorMap &tmA, const CUtensorMap &tmB, const KernelArgs &ka, int grid, cudaStream_t stream) {
    using Cfg = TileCfg<BN>;
    static DeviceOnce configured;
    if (!configured.done()) {
        int rc = cuda_check(cudaFuncSetAttribute(gemm_tc_kernel<BN, LN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 Cfg::SMEM_BYTES), "gemm: shared memory opt-in");
        if (rc) return rc;
        configured.set();
    }
    return cuda_check(launch_pdl(gemm_tc_kernel<BN, LN>, dim3(grid), dim3(NUM_THREADS), Cfg::SMEM_BYTES, stream, tmA, tmB, ka),
                      "gemm: launch");
}

template <int BN>
int launch_bn(const CUtensorMap &tmA, const CUtensorMap &tmB, const KernelArgs &ka, int grid, cudaStream_t stream) {
    return ka.epi.ln_out ? launch_bn_as<BN, true>(tmA, tmB, ka, grid, stream)
                         : launch_bn_as<BN, false>(tmA, tmB, ka, grid, stream);
}

}  // namespace

int gemm_pick_bn(const GemmShape &s) {
    const int sms = sm_count() > 0 ? sm_count() : 148;
    const long long tiles_m = (s.m + BM - 1) / BM;
    const bool pairs_ok = true;
    // CTA pairs on 256 x 256 tiles when that gives every pair of SMs about two work items
    const long long pair_items = ((s.m + 2 * BM - 1) / (2 * BM)) * ((s.n_out + BN2 - 1) / BN2) * s.groups;
    if (pair_items >= sms && pairs_ok) return GEMM_TILE_PAIR;
    // Fewer tiles: the tile width decides how many rounds the SMs need, and a round costs about its width plus a
    // fixed part (the A tile, set-up, drain).  156 tiles of 64 columns are two rounds on 148 SMs where 104 tiles
    // of 96 columns are one.
    int best = 64;
    long long best_cost = -1;
    for (int bn = 256; bn >= 32; bn -= 32) {
        const long long items = tiles_m * ((s.n_out + bn - 1) / bn) * s.groups;
        const long long rounds = (items + sms - 1) / sms;
        const long long cost = rounds * (bn + 64);
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            best = bn;
        }
    }
    // A pair's 256 x 256 tile is a 128 x 256 tile per SM that needs a third less operand fill, measured 0.92 of the
    // single CTA's time at equal rounds (4 x 1024 x 1024 x 1024: 15.5 against 16.9 us; 4 x 512 x 2496 x 4992:
    // 64.6 against 75.3).  Not with a single M tile, where half of every pair would idle.
    if (pairs_ok && s.m > BM) {
        const long long pair_rounds = (pair_items + sms / 2 - 1) / (sms / 2);
        if (pair_rounds * 295 < best_cost) return GEMM_TILE_PAIR;
    }
    return best;
}

int gemm_encode_a(CUtensorMap *map, const GemmOperands &op, const GemmShape &s) {
    const bool shared = op.a_gstride == 0 || s.groups == 1;
    return encode_tma_3d_bf16(map, op.a, s.k, s.m, shared ? 1 : s.groups, op.lda,
                              shared ? (uint64_t)op.lda * s.m : (uint64_t)op.a_gstride, BK, BM);
}

int gemm_encode_b(CUtensorMap *map, const GemmOperands &op, const GemmShape &s, int bn) {
    if (bn == GEMM_TILE_PAIR) bn = BN2 / 2;  // each CTA of a pair loads half of the 256-row W tile
    const bool shared = op.w_gstride == 0 || s.groups == 1;
    return encode_tma_3d_bf16(map, op.w, s.k, s.n_out, shared ? 1 : s.groups, op.ldw,
                              shared ? (uint64_t)op.ldw * s.n_out : (uint64_t)op.w_gstride, BK, bn);
}

int launch_gemm_tc(const GemmOperands &op, const GemmShape &s, const EpiParams &epi, const CUtensorMap *tmA,
                   const CUtensorMap *tmB, int b_g0, int bn_hint, uint32_t *d_status, cudaStream_t stream) {
    if (s.groups < 1 || s.m < 1 || s.n_out < 1 || s.k < 8) return KRAKEN_EINVAL;
    if ((op.lda & 7) || (op.ldw & 7) || (reinterpret_cast<uintptr_t>(op.a) & 15) ||
        (reinterpret_cast<uintptr_t>(op.w) & 15) || (op.a_gstride & 7) || (op.w_gstride & 7))
        return KRAKEN_EUNSUPPORTED;
    const int bn = bn_hint ? bn_hint : gemm_pick_bn(s);
    CUtensorMap la, lb;
    if (!tmA) {
        int rc = gemm_encode_a(&la, op, s);
        if (rc) return rc;
        tmA = &la;
    }
    if (!tmB) {
        int rc = gemm_encode_b(&lb, op, s, bn);
        if (rc) return rc;
        tmB = &lb;
    }
    KernelArgs ka;
    ka.shape = s;
    ka.epi = epi;
    ka.tiles_m = (s.m + BM - 1) / BM;
    const int bn_cols = bn == GEMM_TILE_PAIR ? BN2 : bn;
    ka.tiles_n = (s.n_out + bn_cols - 1) / bn_cols;
    ka.a_gmul = (op.a_gstride == 0 || s.groups == 1) ? 0 : 1;
    ka.b_gmul = (op.w_gstride == 0 || s.groups == 1) ? 0 : 1;
    ka.a_g0 = 0;
    ka.b_g0 = b_g0;
    ka.group_serial = epi.kind == KRAKEN_EPI_RESID_SUM ? 1 : 0;
    ka.n_fastest = (ka.group_serial && ka.tiles_n <= ka.tiles_m) ? 1 : 0;
    if (epi.ln_out) {
        // LayerNorm behind the epilogue: the N tiles of a row block wait for each other, so they must be in
        // flight together: N tiles run fastest (neighbouring CTAs take one row block), and a row block may not be
        // wider than the grid
        if (epi.kind != KRAKEN_EPI_RESID_F32 && epi.kind != KRAKEN_EPI_RESID_SUM) return KRAKEN_EINVAL;
        if (!epi.ln_gamma || !epi.ln_parts || !epi.ln_cnt || !epi.resid || !epi.out_f32) return KRAKEN_EINVAL;
        ka.epi.ln_n_parts = 2 * ka.tiles_n;
        ka.n_fastest = 1;
        const int sms_ = sm_count() > 0 ? sm_count() : 148;
        if (ka.tiles_n > (bn == GEMM_TILE_PAIR ? sms_ / 2 : sms_)) return KRAKEN_EUNSUPPORTED;
    }
    ka.w_early = op.w_static ? 1 : 0;
    ka.status = d_status;
    if (bn == GEMM_TILE_PAIR)
        return epi.ln_out ? launch_pair<true>(*tmA, *tmB, ka, stream) : launch_pair<false>(*tmA, *tmB, ka, stream);
    const long long tiles = (long long)ka.tiles_m * ka.tiles_n;
    const long long units = ka.group_serial ? tiles : tiles * s.groups;
    const int sms = sm_count() > 0 ? sm_count() : 148;
    int grid = static_cast<int>(units < sms ? units : sms);
    if (epi.ln_out && grid > ka.tiles_n) grid -= grid % ka.tiles_n;   // whole row blocks per round, as for the pairs
    switch (bn) {
        case 256: return launch_bn<256>(*tmA, *tmB, ka, grid, stream);
        case 224: return launch_bn<224>(*tmA, *tmB, ka, grid, stream);
        case 192: return launch_bn<192>(*tmA, *tmB, ka, grid, stream);
        case 160: return launch_bn<160>(*tmA, *tmB, ka, grid, stream);
        case 128: return launch_bn<128>(*tmA, *tmB, ka, grid, stream);
        case 96: return launch_bn<96>(*tmA, *tmB, ka, grid, stream);
        case 64: return launch_bn<64>(*tmA, *tmB, ka, grid, stream);
        case 32: return launch_bn<32>(*tmA, *tmB, ka, grid, stream);
        default: return KRAKEN_EINVAL;
    }
}

size_t gemm_ln_parts_bytes(int groups, int m, int n_out, int bn) {
    const int cols = bn == GEMM_TILE_PAIR ? BN2 : bn;
    return (size_t)groups * m * 2 * ((n_out + cols - 1) / cols) * sizeof(float4);
}

size_t gemm_ln_cnt_bytes(int groups, int m) { return (size_t)groups * ln_slabs(m) * 2 * sizeof(uint32_t); }

}  // namespace kr
