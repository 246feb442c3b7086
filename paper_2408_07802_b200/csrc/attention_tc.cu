// Causal prefill attention on the sm_100a tensor cores (tcgen05 + TMEM), one CTA per tile of 128
// query rows of one (branch, sequence, head), streaming K/V tiles of 128 keys by TMA.
//
//   warp 0      TMA producer: Q once, then K and V tiles into two-stage rings (128-byte swizzle);
//   warp 1      MMA issuer:   S_j = Q K_j^T  (both operands K-major in shared memory) into one of two
//                             S buffers in TMEM, then O_j = P_j V_j with P_j read from TMEM (it
//                             overwrites S_j in place as packed bf16) and V_j MN-major in shared memory;
//   warps 2-5   softmax:      one thread per query row (TMEM lane = row, so row max and row sum need
//                             no shuffles): tcgen05.ld of S_j, causal mask, exp2 with the scale folded
//                             in, tcgen05.st of P_j, then the running output kept in registers
//                             acc = acc * corr + O_j  with O_j fetched from TMEM.
// S_{j+1} = Q K_{j+1}^T is issued before P_j V_j, so the tensor pipe works on the next scores while
// the softmax warps are busy with the current ones.  TMEM: 2 x 128 columns of S/P, 2 x HD of O_j.
// Every mbarrier wait is time-bounded and falls through to a common teardown.
#include <math.h>

#include "internal.h"
#include "ptx.cuh"

namespace kr {

namespace {

constexpr int TQ = 128;   // query rows per CTA
constexpr int TK = 128;   // keys per tile
constexpr int ATC_THREADS = 192;

struct AttnTcArgs {
    int groups, batch, seqlen, pos0, n_head;
    uint16_t *out;
    long long out_gstride;
    uint32_t *status;
};

__device__ __forceinline__ void tmem_ld_32x32_nowait(uint32_t taddr, uint32_t (&r)[32]) { tmem_ld_32x32(taddr, r); }

// 32 lanes x 16 columns store
__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

// MN-major operand (V: rows = keys, 64 head-dim columns = 128 bytes per row, 128-byte swizzle):
// groups of 8 keys are 1024 bytes apart (stride byte offset); the next 64 columns of the head
// dimension live in a separate tile `lbo_bytes` further (leading byte offset).
__device__ __forceinline__ uint64_t umma_desc_sw128_mnmajor(uint32_t smem_addr, uint32_t lbo_bytes) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= static_cast<uint64_t>(1024 >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(2) << 61;
    return d;
}

template <int HD>
struct AtcCfg {
    static constexpr int HALVES = HD / 64;                 // 64-column (128-byte) pieces of the head dim
    static constexpr int TILE_BYTES = TK * 128;            // one 128 x 64 bf16 piece
    static constexpr int Q_BYTES = HALVES * TILE_BYTES;
    static constexpr int KV_BYTES = HALVES * TILE_BYTES;   // one K (or V) tile
    static constexpr int STAGES = 2;
    static constexpr int SMEM_BYTES = Q_BYTES + 2 * STAGES * KV_BYTES + 1024 + 256;
    static constexpr int S_COL0 = 0;                       // S buffers at columns 0 and 128
    static constexpr int O_COL0 = 256;                     // O buffers at 256 and 256 + HD
    static constexpr int TMEM_COLS = 512;
};

template <int HD>
__global__ void __launch_bounds__(ATC_THREADS, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const AttnTcArgs a) {
    using Cfg = AtcCfg<HD>;
    extern __shared__ uint8_t smem_raw_atc[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw_atc) + 1023) & ~uintptr_t(1023));
    uint8_t *sQ = smem;
    uint8_t *sK = sQ + Cfg::Q_BYTES;                       // [STAGES][KV_BYTES]
    uint8_t *sV = sK + Cfg::STAGES * Cfg::KV_BYTES;        // [STAGES][KV_BYTES]
    uint64_t *bars = reinterpret_cast<uint64_t *>(sV + Cfg::STAGES * Cfg::KV_BYTES);
    uint64_t *q_full = bars;            // 1
    uint64_t *k_full = bars + 1;        // [2]
    uint64_t *k_empty = bars + 3;       // [2]
    uint64_t *v_full = bars + 5;        // [2]
    uint64_t *v_empty = bars + 7;       // [2]
    uint64_t *s_full = bars + 9;        // [2]  scores ready            (MMA -> softmax)
    uint64_t *p_ready = bars + 11;      // [2]  probabilities in TMEM   (softmax -> MMA)
    uint64_t *o_full = bars + 13;       // [2]  P V product ready       (MMA -> softmax)
    uint64_t *o_empty = bars + 15;      // [2]  product consumed        (softmax -> MMA)
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 17);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int mt = gridDim.x - 1 - blockIdx.x;             // longest rows first
    const int h = blockIdx.y;
    const int b = blockIdx.z % a.batch, g = blockIdx.z / a.batch;
    const int q0 = mt * TQ;
    const int rows_valid = min(TQ, a.seqlen - q0);
    const int n_keys = a.pos0 + q0 + rows_valid;           // keys visible to the last valid row
    const int n_tiles = (n_keys + TK - 1) / TK;

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(k_full + s, 1);
            mbar_init(k_empty + s, 1);
            mbar_init(v_full + s, 1);
            mbar_init(v_empty + s, 1);
            mbar_init(s_full + s, 1);
            mbar_init(p_ready + s, 4);
            mbar_init(o_full + s, 1);
            mbar_init(o_empty + s, 4);
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tmQ);
        prefetch_tensormap(&tmK);
        prefetch_tensormap(&tmV);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // Q: rows of this sequence's tile, columns of this head
            mbar_expect_tx(q_full, Cfg::Q_BYTES);
#pragma unroll
            for (int hf = 0; hf < Cfg::HALVES; ++hf)
                tma_load_3d(sQ + hf * Cfg::TILE_BYTES, &tmQ, q_full, h * HD + hf * 64, b * a.seqlen + q0, g);
            bool ok = true;
            for (int j = 0; ok && j < n_tiles; ++j) {
                const int st = j & 1;
                const uint32_t ph = (j >> 1) & 1;
                if (!(ok = mbar_wait(k_empty + st, ph ^ 1u, abort_flag))) break;
                mbar_expect_tx(k_full + st, Cfg::KV_BYTES);
#pragma unroll
                for (int hf = 0; hf < Cfg::HALVES; ++hf)
                    tma_load_4d(sK + st * Cfg::KV_BYTES + hf * Cfg::TILE_BYTES, &tmK, k_full + st, hf * 64, j * TK,
                                b * a.n_head + h, g);
                if (!(ok = mbar_wait(v_empty + st, ph ^ 1u, abort_flag))) break;
                mbar_expect_tx(v_full + st, Cfg::KV_BYTES);
#pragma unroll
                for (int hf = 0; hf < Cfg::HALVES; ++hf)
                    tma_load_4d(sV + st * Cfg::KV_BYTES + hf * Cfg::TILE_BYTES, &tmV, v_full + st, hf * 64, j * TK,
                                b * a.n_head + h, g);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc_qk = umma_idesc_bf16(TQ, TK);
            constexpr uint32_t idesc_pv = umma_idesc_bf16(TQ, HD) | (1u << 16);  // B (V) is MN-major
            bool ok = mbar_wait(q_full, 0, abort_flag);
            const uint32_t q_addr = smem_u32(sQ);
            auto issue_qk = [&](int j) -> bool {
                const int st = j & 1;
                if (!mbar_wait(k_full + st, (j >> 1) & 1, abort_flag)) return false;
                tc_fence_after_sync();
                const uint32_t k_addr = smem_u32(sK + st * Cfg::KV_BYTES);
                const uint32_t d_tmem = tmem_base + Cfg::S_COL0 + st * TK;
#pragma unroll
                for (int ks = 0; ks < HD / 16; ++ks) {
                    const uint32_t off = (ks >> 2) * Cfg::TILE_BYTES + (ks & 3) * 32;
                    umma_bf16_ss(d_tmem, umma_desc_sw128_kmajor(q_addr + off), umma_desc_sw128_kmajor(k_addr + off),
                                 idesc_qk, ks != 0 ? 1u : 0u);
                }
                umma_commit(k_empty + st);
                umma_commit(s_full + st);
                return true;
            };
            if (ok) ok = issue_qk(0);
            for (int j = 0; ok && j < n_tiles; ++j) {
                const int st = j & 1;
                const uint32_t ph = (j >> 1) & 1;
                if (j + 1 < n_tiles && !(ok = issue_qk(j + 1))) break;
                if (!(ok = mbar_wait(p_ready + st, ph, abort_flag))) break;
                if (!(ok = mbar_wait(v_full + st, ph, abort_flag))) break;
                if (!(ok = mbar_wait(o_empty + st, ph ^ 1u, abort_flag))) break;
                tc_fence_after_sync();
                const uint32_t v_addr = smem_u32(sV + st * Cfg::KV_BYTES);
                const uint32_t p_tmem = tmem_base + Cfg::S_COL0 + st * TK;
                const uint32_t o_tmem = tmem_base + Cfg::O_COL0 + st * HD;
#pragma unroll
                for (int ks = 0; ks < TK / 16; ++ks) {
                    // 16 keys per step: 8 packed columns of P, two 8-key groups (2 x 1024 bytes) of V
                    umma_bf16_ts(o_tmem, p_tmem + ks * 8,
                                 umma_desc_sw128_mnmajor(v_addr + ks * 2048, Cfg::TILE_BYTES), idesc_pv,
                                 ks != 0 ? 1u : 0u);
                }
                umma_commit(v_empty + st);
                umma_commit(o_full + st);
            }
        }
        __syncwarp();
    } else {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;                 // row of the tile = TMEM lane
        const int qpos = a.pos0 + q0 + row;                  // position of this query
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const float sl2 = rsqrtf(static_cast<float>(HD)) * 1.4426950408889634f;
        float acc[HD];
#pragma unroll
        for (int i = 0; i < HD; ++i) acc[i] = 0.f;
        float m = -INFINITY, l = 0.f;
        bool ok = true;

        auto add_product = [&](int j) -> bool {              // acc += O_j
            const int st = j & 1;
            bool good = mbar_wait(o_full + st, (j >> 1) & 1, abort_flag);
            good = __all_sync(0xFFFFFFFFu, good);
            if (!good) return false;
            tc_fence_after_sync();
#pragma unroll
            for (int c = 0; c < HD / 32; ++c) {
                uint32_t r[32];
                tmem_ld_32x32(lane_addr + Cfg::O_COL0 + st * HD + c * 32, r);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) acc[c * 32 + i] += __uint_as_float(r[i]);
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(o_empty + st);
            return true;
        };

        for (int j = 0; j < n_tiles; ++j) {
            const int st = j & 1;
            ok = mbar_wait(s_full + st, (j >> 1) & 1, abort_flag);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t s_addr = lane_addr + Cfg::S_COL0 + st * TK;
            const bool diag = j * TK + TK - 1 > a.pos0 + q0;  // tile may hold keys beyond some query of this CTA
            // pass 1: row maximum
            float mx = -INFINITY;
#pragma unroll
            for (int c = 0; c < TK / 32; ++c) {
                uint32_t r[32];
                tmem_ld_32x32(s_addr + c * 32, r);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    float s = __uint_as_float(r[i]);
                    if (diag && j * TK + c * 32 + i > qpos) s = -INFINITY;
                    mx = fmaxf(mx, s);
                }
            }
            const float m_new = fmaxf(m, mx);                 // finite: key 0 is visible to every query
            const float corr = ex2_approx((m - m_new) * sl2);
            const float ms = m_new * sl2;
            // pass 2: probabilities, packed to bf16 over the scores they came from
            float sum = 0.f;
#pragma unroll
            for (int c = 0; c < TK / 32; ++c) {
                uint32_t r[32];
                tmem_ld_32x32(s_addr + c * 32, r);
                tmem_ld_wait();
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    float s0 = __uint_as_float(r[2 * i]), s1 = __uint_as_float(r[2 * i + 1]);
                    if (diag) {
                        if (j * TK + c * 32 + 2 * i > qpos) s0 = -INFINITY;
                        if (j * TK + c * 32 + 2 * i + 1 > qpos) s1 = -INFINITY;
                    }
                    const float p0 = ex2_approx(fmaf(s0, sl2, -ms));
                    const float p1 = ex2_approx(fmaf(s1, sl2, -ms));
                    sum += p0 + p1;
                    pk[i] = pack_bf16x2(p0, p1);
                }
                tmem_st_32x16(s_addr + c * 16, pk);
            }
            tmem_st_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_ready + st);
            l = l * corr + sum;
            if (j > 0 && !(ok = add_product(j - 1))) break;
#pragma unroll
            for (int i = 0; i < HD; ++i) acc[i] *= corr;
            m = m_new;
        }
        if (ok && n_tiles > 0) ok = add_product(n_tiles - 1);
        if (ok && row < rows_valid) {
            const float inv = 1.f / l;
            const int d = a.n_head * HD;
            uint16_t *dst = a.out + g * a.out_gstride + ((long long)b * a.seqlen + q0 + row) * d + h * HD;
#pragma unroll
            for (int i = 0; i < HD / 8; ++i) {
                uint4 u;
                u.x = pack_bf16x2(acc[8 * i + 0] * inv, acc[8 * i + 1] * inv);
                u.y = pack_bf16x2(acc[8 * i + 2] * inv, acc[8 * i + 3] * inv);
                u.z = pack_bf16x2(acc[8 * i + 4] * inv, acc[8 * i + 5] * inv);
                u.w = pack_bf16x2(acc[8 * i + 6] * inv, acc[8 * i + 7] * inv);
                reinterpret_cast<uint4 *>(dst)[i] = u;
            }
        }
    }

    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
        if (threadIdx.x == 0 && a.status) atomicOr(a.status, STATUS_WAIT_LIMIT);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
}

template <int HD>
int launch(const CUtensorMap &tmQ, const CUtensorMap &tmK, const CUtensorMap &tmV, const AttnTcArgs &a,
           cudaStream_t stream) {
    using Cfg = AtcCfg<HD>;
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(attn_tc_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES) !=
            cudaSuccess)
            return KRAKEN_ECUDA;
        configured = true;
    }
    dim3 grid((a.seqlen + TQ - 1) / TQ, a.n_head, a.batch * a.groups);
    attn_tc_kernel<HD><<<grid, ATC_THREADS, Cfg::SMEM_BYTES, stream>>>(tmQ, tmK, tmV, a);
    return cudaGetLastError() == cudaSuccess ? KRAKEN_OK : KRAKEN_ECUDA;
}

}  // namespace

bool attention_tc_supported(const AttnParams &p) {
    if (p.head_dim != 64 && p.head_dim != 128) return false;
    // the cache of one group must be [batch][head][max_pos][head_dim] without gaps
    if (p.cache_bstride != (long long)p.n_head * p.max_pos * p.head_dim) return false;
    const int d = p.n_head * p.head_dim;
    if ((reinterpret_cast<uintptr_t>(p.q) & 15) || (reinterpret_cast<uintptr_t>(p.k_cache) & 15) ||
        (reinterpret_cast<uintptr_t>(p.v_cache) & 15) || (reinterpret_cast<uintptr_t>(p.out) & 15) ||
        (p.q_gstride & 7) || (p.cache_gstride & 7) || (p.out_gstride & 7) || (d & 7))
        return false;
    return true;
}

int attention_tc_encode(const AttnParams &p, CUtensorMap *tmQ, CUtensorMap *tmK, CUtensorMap *tmV) {
    const int d = p.n_head * p.head_dim;
    const long long T = (long long)p.batch * p.seqlen;
    const bool one = p.groups == 1;
    int rc = encode_tma_3d_bf16(tmQ, p.q, d, T, p.groups, d, one ? (uint64_t)T * d : (uint64_t)p.q_gstride, 64, TQ);
    if (rc) return rc;
    // rows past the keys written so far are out of bounds of the map and read as zeros
    const uint64_t kv_len = (uint64_t)p.pos0 + p.seqlen;
    const uint64_t dims[4] = {(uint64_t)p.head_dim, kv_len, (uint64_t)p.batch * p.n_head, (uint64_t)p.groups};
    const uint64_t strides[3] = {(uint64_t)p.head_dim, (uint64_t)p.max_pos * p.head_dim,
                                 one ? (uint64_t)p.cache_bstride * p.batch : (uint64_t)p.cache_gstride};
    const uint32_t box[4] = {64, TK, 1, 1};
    rc = encode_tma_4d_bf16(tmK, p.k_cache, dims, strides, box);
    if (rc) return rc;
    return encode_tma_4d_bf16(tmV, p.v_cache, dims, strides, box);
}

int launch_attention_tc(const AttnParams &p, const CUtensorMap *tmQ, const CUtensorMap *tmK, const CUtensorMap *tmV,
                        uint32_t *d_status, cudaStream_t stream) {
    if (!p.q || !p.k_cache || !p.v_cache || !p.out || p.groups < 1 || p.batch < 1 || p.seqlen < 1 || p.pos0 < 0 ||
        p.n_head < 1 || p.pos0 + p.seqlen > p.max_pos)
        return KRAKEN_EINVAL;
    if (!attention_tc_supported(p)) return KRAKEN_EUNSUPPORTED;
    CUtensorMap lq, lk, lv;
    if (!tmQ || !tmK || !tmV) {
        int rc = attention_tc_encode(p, &lq, &lk, &lv);
        if (rc) return rc;
        tmQ = &lq;
        tmK = &lk;
        tmV = &lv;
    }
    AttnTcArgs a;
    a.groups = p.groups;
    a.batch = p.batch;
    a.seqlen = p.seqlen;
    a.pos0 = p.pos0;
    a.n_head = p.n_head;
    a.out = p.out;
    a.out_gstride = p.out_gstride;
    a.status = d_status;
    return p.head_dim == 64 ? launch<64>(*tmQ, *tmK, *tmV, a, stream) : launch<128>(*tmQ, *tmK, *tmV, a, stream);
}

}  // namespace kr
