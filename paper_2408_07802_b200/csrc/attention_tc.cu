// Causal prefill attention on the sm_100a tensor cores (tcgen05 + TMEM).
//
// One CTA owns TWO tiles of 128 query rows of one (branch, sequence, head) and streams K/V tiles of
// 128 keys by TMA; the two query tiles share every K/V tile and take turns on the tensor pipe, so
// that while one tile's scores are in the softmax the other tile's matrix products run.
//
//   warp 0      TMA producer: both Q tiles once, then K and V tiles into a two-stage ring whose stage
//               holds what one step of the issuer reads, V_j and K_{j+1} (one barrier wait and one release
//               per step; 128-byte swizzle; rows past the keys written so far are out of bounds = zeros);
//   warp 1      MMA issuer, per K/V tile j and query tile w:
//                   S_w = Q_w K_j^T          both operands K-major in shared memory -> TMEM
//                   O_w (+)= P_w V_j         P_w read from TMEM (packed 16-bit), V_j MN-major in shared memory,
//                                            O_w accumulates in TMEM
//               With 128-wide O tensor memory is full and P_w overwrites S_w in place: the products are issued in
//               the order PV_0(j), QK_0(j+1), PV_1(j), QK_1(j+1).  With head dims up to 64 P_w has columns of its
//               own and the order is QK_0(j+1), QK_1(j+1) as soon as the softmax warps hold S_w(j) in registers,
//               then PV_0(j), PV_1(j): the softmax of a query tile never waits for its next scores
//               (64 heads x 1024 tokens 34.9 -> 31.2 us, 16 x 64 heads x 2048 tokens 1080 -> 1006 us);
//   warps 2-5   softmax of query tile 0, warps 6-9 of query tile 1: one thread per query row (TMEM
//               lane = row: row max and row sum need no shuffles).  The whole score row is pulled into
//               registers with tcgen05.ld, masked on diagonal tiles, exponentiated with the scale folded
//               into one packed FMA, stored back as P with tcgen05.st.
// The running maximum is only raised when a row's new maximum exceeds the one in use by more than
// 2^8 in the exponent; then (rarely) the warp rescales its rows of O in TMEM before releasing P.
// Using a stale maximum is exact: numerator and denominator carry the same factor.
// Every role walks a list of work items with running barrier phases, so a CTA can take several items
// without draining its pipeline: with enough work each SM gets one CTA and a fixed list of couples of items
// of equal total length (atc_next), else the grid has one CTA per item (see launch()).
// TMEM: head dim 128: S/P of tile w at column 128 w, O of tile w at 256 + 128 w; head dim 64: S at 128 w, P at
// 256 + 64 w, O at 384 + 64 w.  All waits are time-bounded.  Exponentials as a polynomial on the FMA pipe (a quarter
// or half of them) measured slower in both layouts (1241 / 1276 against 1006 us): the softmax warps are bound by
// instruction issue, not by the exp unit.
#include <math.h>

#include "internal.h"
#include "ptx.cuh"

namespace kr {

namespace {

constexpr int TQ = 128;   // query rows per tile (two tiles per CTA)
constexpr int TK = 128;   // keys per tile
constexpr int ATC_THREADS = 320;
constexpr float RESCALE_LOG2 = 8.0f;
struct AttnTcArgs {
    int groups, batch, seqlen, pos0, n_head;
    int n_kv_head, kv_rep;   // key/value heads in the cache; query heads per key/value head
    int balanced;            // 1: a fixed list of work per CTA, built from pairs of items of equal total length
    int head_dim;      // <= HD of the kernel instance, a multiple of 8 (columns past it are zero-filled by TMA)
    uint16_t *out;
    long long out_gstride;
    uint32_t *status;
};

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

// 32 lanes x 16 columns store
__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

__device__ __forceinline__ float max3f(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// (x0, x1) * a + b on the packed fp32 pipe
__device__ __forceinline__ void fma2(float &x0, float &x1, float a, float b) {
    asm("{\n"
        ".reg .b64 rx, ra, rb;\n"
        "mov.b64 rx, {%0, %1};\n"
        "mov.b64 ra, {%2, %2};\n"
        "mov.b64 rb, {%3, %3};\n"
        "fma.rn.f32x2 rx, rx, ra, rb;\n"
        "mov.b64 {%0, %1}, rx;\n"
        "}\n"
        : "+f"(x0), "+f"(x1)
        : "f"(a), "f"(b));
}

template <int HD>
struct AtcCfg {
    static constexpr int HALVES = HD / 64;                 // 64-column (128-byte) pieces of the head dim
    static constexpr int TILE_BYTES = TK * 128;            // one 128 x 64 bf16 piece
    static constexpr int Q_BYTES = HALVES * TILE_BYTES;    // one Q tile
    static constexpr int KV_BYTES = HALVES * TILE_BYTES;   // one K (or V) tile
    static constexpr int STAGES = 2;
    static constexpr int BUNDLE_BYTES = 2 * KV_BYTES;      // a ring stage: V_j, then K_{j+1}
    static constexpr int SMEM_BYTES = 2 * Q_BYTES + STAGES * BUNDLE_BYTES + 1024 + 256;
    static constexpr int S_COL0 = 0;                       // S of query tile w at 128 w
    // Head dims up to 64 leave tensor-memory columns free (O is 64 wide): P then gets columns of its own, so the
    // next scores of a query tile are issued as soon as its softmax warps hold the current ones in registers,
    // instead of after the product that reads P.  With 128-wide O the 512 columns are full and P overwrites S.
    static constexpr bool SEPARATE_P = HD <= 64;
    static constexpr int P_COLS = TK / 2;                  // packed 16-bit probabilities of one tile
    static constexpr int P_COL0 = SEPARATE_P ? 256 : S_COL0;
    static constexpr int P_STRIDE = SEPARATE_P ? P_COLS : TK;
    static constexpr int O_COL0 = SEPARATE_P ? 384 : 256;  // O of query tile w at O_COL0 + HD w (128 w when P overwrites S)
    static constexpr int O_STRIDE = SEPARATE_P ? HD : TK;
    static constexpr int TMEM_COLS = 512;
};

// A work item is one pair of query tiles of one (branch, sequence, head).  Items of one head are
// neighbours in the order (their K/V tiles meet in L2), longest pair first.
struct AtcItem {
    int q0, h, b, g;
    int n_tiles[2];
    int n_max;
};

__device__ __forceinline__ bool atc_item(const AttnTcArgs &a, int idx, AtcItem &it) {
    const int n_pairs = (a.seqlen + 2 * TQ - 1) / (2 * TQ);
    const long long total = (long long)n_pairs * a.n_head * a.batch * a.groups;
    if (idx >= total) return false;
    const int pair = n_pairs - 1 - idx % n_pairs;
    const int hb = idx / n_pairs;
    it.h = hb % a.n_head;
    const int bg = hb / a.n_head;
    it.b = bg % a.batch;
    it.g = bg / a.batch;
    it.q0 = pair * 2 * TQ;
#pragma unroll
    for (int w = 0; w < 2; ++w) {
        const int rows = min(TQ, a.seqlen - (it.q0 + w * TQ));
        it.n_tiles[w] = rows > 0 ? (a.pos0 + it.q0 + w * TQ + rows + TK - 1) / TK : 0;
    }
    it.n_max = max(it.n_tiles[0], it.n_tiles[1]);
    return true;
}

// The j-th work item of this CTA (j = 0, 1, ...; advanced here), false when the CTA is done.
//   one CTA per item:  item blockIdx.x only.
//   balanced list:     the work of a causal item grows linearly with its place in the sequence, so the k-th
//                      longest and the k-th shortest pair of query tiles of one head together always cost the
//                      same.  Such couples are dealt round-robin to the CTAs (couple c, c + grid, ...), long
//                      half first, which gives every CTA the same work without a queue, keeps a head's K/V on
//                      neighbouring CTAs, and lets a CTA start the next item while the last one drains.
__device__ __forceinline__ bool atc_next(const AttnTcArgs &a, int &j, AtcItem &it) {
    if (!a.balanced) {
        if (j != 0) return false;
        ++j;
        return atc_item(a, blockIdx.x, it);
    }
    const int n_pairs = (a.seqlen + 2 * TQ - 1) / (2 * TQ);
    const int couples = (n_pairs + 1) / 2;                    // per head; the middle pair stands alone when odd
    const long long total = (long long)couples * a.n_head * a.batch * a.groups;
    for (;;) {
        const long long c = blockIdx.x + (long long)(j >> 1) * gridDim.x;
        if (c >= total) return false;
        const int k = static_cast<int>(c % couples);
        const int hb = static_cast<int>(c / couples);
        const bool second = j & 1;
        ++j;
        if (second && k == n_pairs - 1 - k) continue;         // the middle pair has no partner
        // atc_item numbers the pairs of a head longest first: index k is the (k+1)-th longest
        return atc_item(a, hb * n_pairs + (second ? n_pairs - 1 - k : k), it);
    }
}

template <int HD>
__global__ void __launch_bounds__(ATC_THREADS, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const AttnTcArgs a) {
    using Cfg = AtcCfg<HD>;
    extern __shared__ uint8_t smem_raw_atc[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw_atc) + 1023) & ~uintptr_t(1023));
    uint8_t *sQ = smem;                                    // [2][Q_BYTES]
    uint8_t *sB = sQ + 2 * Cfg::Q_BYTES;                   // [STAGES][V tile | K tile]
    uint64_t *bars = reinterpret_cast<uint64_t *>(sB + Cfg::STAGES * Cfg::BUNDLE_BYTES);
    uint64_t *q_full = bars;            // 1    Q tiles of the current item loaded
    uint64_t *q_empty = bars + 1;       // 1    every S = Q K^T of the item has finished reading Q
    uint64_t *b_full = bars + 2;        // [2]  V_j and K_{j+1} loaded
    uint64_t *b_empty = bars + 4;       // [2]  every product that reads them has finished
    uint64_t *s_full = bars + 6;        // [2]  scores of query tile w ready      (MMA -> softmax w)
    uint64_t *p_ready = bars + 8;       // [2]  probabilities of tile w in TMEM   (softmax w -> MMA)
    uint64_t *pv_done = bars + 10;      // [2]  O_w of the item is complete       (MMA -> softmax w)
    uint64_t *s_free = bars + 12;       // [2]  scores of tile w are in registers (softmax w -> MMA; separate P only)
    uint64_t *p_free = bars + 14;       // [2]  the product that read P_w is done (MMA -> softmax w; separate P only)
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 16);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        mbar_init(q_empty, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(b_full + s, 1);
            mbar_init(b_empty + s, 1);
            mbar_init(s_full + s, 1);
            mbar_init(p_ready + s, 4);
            mbar_init(pv_done + s, 1);
            mbar_init(s_free + s, 4);
            mbar_init(p_free + s, 1);
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
    pdl_wait();   // launched ahead of the end of its predecessor: nothing of the predecessor's is touched before here
    pdl_trigger();   // the successor's CTAs may take this one's place as soon as it leaves

    // Every role walks the same item sequence (blockIdx.x, + gridDim.x, ...) and keeps running
    // counters for the barrier phases, so the pipeline never drains between items.
    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            uint32_t kv_cnt = 0, item_cnt = 0;
            AtcItem it;
            for (int jj = 0; ok && atc_next(a, jj, it); ++item_cnt) {
                if (!(ok = mbar_wait(q_empty, (item_cnt & 1u) ^ 1u, abort_flag))) break;
                const int q_tiles = it.n_tiles[1] > 0 ? 2 : 1;
                mbar_expect_tx(q_full, q_tiles * Cfg::Q_BYTES);
                for (int w = 0; w < q_tiles; ++w)
#pragma unroll
                    for (int hf = 0; hf < Cfg::HALVES; ++hf)
                        tma_load_3d(sQ + w * Cfg::Q_BYTES + hf * Cfg::TILE_BYTES, &tmQ, q_full, it.h * a.head_dim + hf * 64,
                                    it.b * a.seqlen + it.q0 + w * TQ, it.g);
                // stage -1 of the item holds K_0 alone; stage j holds V_j and, unless it is the last, K_{j+1}
                const int kvh = it.b * a.n_kv_head + it.h / a.kv_rep;
                for (int j = -1; ok && j < it.n_max; ++j, ++kv_cnt) {
                    const int st = kv_cnt & 1;
                    const uint32_t ph = (kv_cnt >> 1) & 1;
                    if (!(ok = mbar_wait(b_empty + st, ph ^ 1u, abort_flag))) break;
                    const bool has_v = j >= 0, has_k = j + 1 < it.n_max;
                    mbar_expect_tx(b_full + st, ((has_v ? 1 : 0) + (has_k ? 1 : 0)) * Cfg::KV_BYTES);
                    uint8_t *sV = sB + st * Cfg::BUNDLE_BYTES, *sK = sV + Cfg::KV_BYTES;
                    if (has_v) {
#pragma unroll
                        for (int hf = 0; hf < Cfg::HALVES; ++hf)
                            tma_load_4d(sV + hf * Cfg::TILE_BYTES, &tmV, b_full + st, hf * 64, j * TK, kvh, it.g);
                    }
                    if (has_k) {
#pragma unroll
                        for (int hf = 0; hf < Cfg::HALVES; ++hf)
                            tma_load_4d(sK + hf * Cfg::TILE_BYTES, &tmK, b_full + st, hf * 64, (j + 1) * TK, kvh, it.g);
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            // head dims below HD: the scores need ceil(head_dim / 16) steps (K is zero beyond head_dim, so
            // whatever Q holds there does not count), the output ceil(head_dim / 16) * 16 columns
            const int qk_steps = (a.head_dim + 15) / 16;
            constexpr uint32_t idesc_qk = umma_idesc_h16(TQ, TK);
            const uint32_t idesc_pv = umma_idesc_h16(TQ, qk_steps * 16) | (1u << 16);  // B (V) is MN-major
            auto issue_qk = [&](int w, int st) {
                const uint32_t q_addr = smem_u32(sQ + w * Cfg::Q_BYTES);
                const uint32_t k_addr = smem_u32(sB + st * Cfg::BUNDLE_BYTES + Cfg::KV_BYTES);
                const uint32_t d_tmem = tmem_base + Cfg::S_COL0 + w * TK;
#pragma unroll
                for (int ks = 0; ks < HD / 16; ++ks) {
                    if (ks >= qk_steps) break;
                    const uint32_t off = (ks >> 2) * Cfg::TILE_BYTES + (ks & 3) * 32;
                    umma_bf16_ss(d_tmem, umma_desc_sw128_kmajor(q_addr + off), umma_desc_sw128_kmajor(k_addr + off),
                                 idesc_qk, ks != 0 ? 1u : 0u);
                }
                umma_commit(s_full + w);
            };
            auto issue_pv = [&](int w, int st, bool first, bool last) {
                const uint32_t v_addr = smem_u32(sB + st * Cfg::BUNDLE_BYTES);
                const uint32_t p_tmem = tmem_base + Cfg::P_COL0 + w * Cfg::P_STRIDE;
                const uint32_t o_tmem = tmem_base + Cfg::O_COL0 + w * Cfg::O_STRIDE;
#pragma unroll
                for (int ks = 0; ks < TK / 16; ++ks) {
                    // 16 keys per step: 8 packed columns of P, two 8-key groups (2 x 1024 bytes) of V
                    umma_bf16_ts(o_tmem, p_tmem + ks * 8,
                                 umma_desc_sw128_mnmajor(v_addr + ks * 2048, Cfg::TILE_BYTES), idesc_pv,
                                 (first && ks == 0) ? 0u : 1u);
                }
                // the softmax warps need no signal for the products in between: the scores they wait for next
                // are committed after this product, and a commit covers everything issued before it
                if (last) umma_commit(pv_done + w);
                else if (Cfg::SEPARATE_P) umma_commit(p_free + w);   // the softmax may write the next P
            };
            bool ok = true;
            uint32_t kv_cnt = 0, item_cnt = 0, tile_cnt[2] = {0, 0};
            AtcItem it;
            for (int jj = 0; ok && atc_next(a, jj, it); ++item_cnt) {
                if (!(ok = mbar_wait(q_full, item_cnt & 1u, abort_flag))) break;
                if (!(ok = mbar_wait(b_full + (kv_cnt & 1), (kv_cnt >> 1) & 1, abort_flag))) break;
                tc_fence_after_sync();
                if (it.n_tiles[0] > 0) issue_qk(0, kv_cnt & 1);
                if (it.n_tiles[1] > 0) issue_qk(1, kv_cnt & 1);
                umma_commit(b_empty + (kv_cnt & 1));
                ++kv_cnt;
                if (it.n_max == 1) umma_commit(q_empty);
                for (int j = 0; ok && j < it.n_max; ++j, ++kv_cnt) {
                    const int st = kv_cnt & 1;
                    if (!(ok = mbar_wait(b_full + st, (kv_cnt >> 1) & 1, abort_flag))) break;
                    if (Cfg::SEPARATE_P) {
                        // the next scores first: S_w is free as soon as its softmax warps have read it
#pragma unroll
                        for (int w = 0; w < 2; ++w) {
                            if (j + 1 < it.n_tiles[w]) {
                                if (!(ok = mbar_wait(s_free + w, tile_cnt[w] & 1u, abort_flag))) break;
                                tc_fence_after_sync();
                                issue_qk(w, st);
                            }
                        }
                        if (!ok) break;
#pragma unroll
                        for (int w = 0; w < 2; ++w) {
                            if (j < it.n_tiles[w]) {
                                if (!(ok = mbar_wait(p_ready + w, tile_cnt[w] & 1u, abort_flag))) break;
                                ++tile_cnt[w];
                                tc_fence_after_sync();
                                issue_pv(w, st, j == 0, j + 1 == it.n_tiles[w]);
                            }
                        }
                    } else {
#pragma unroll
                        for (int w = 0; w < 2; ++w) {
                            if (j < it.n_tiles[w]) {
                                if (!(ok = mbar_wait(p_ready + w, tile_cnt[w] & 1u, abort_flag))) break;
                                ++tile_cnt[w];
                                tc_fence_after_sync();
                                issue_pv(w, st, j == 0, j + 1 == it.n_tiles[w]);
                            }
                            if (j + 1 < it.n_tiles[w]) issue_qk(w, st);
                        }
                    }
                    if (!ok) break;
                    umma_commit(b_empty + st);
                    if (j + 2 == it.n_max) umma_commit(q_empty);   // the item's last scores are issued
                }
            }
        }
        __syncwarp();
    } else {
        const int w = (warp - 2) >> 2;                       // query tile of this warp
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;                 // row of the tile = TMEM lane
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const uint32_t s_addr = lane_addr + Cfg::S_COL0 + w * TK;
        const uint32_t p_addr = lane_addr + Cfg::P_COL0 + w * Cfg::P_STRIDE;
        const uint32_t o_addr = lane_addr + Cfg::O_COL0 + w * Cfg::O_STRIDE;
        const float sl2 = rsqrtf(static_cast<float>(a.head_dim)) * 1.4426950408889634f;
        bool ok = true;
        uint32_t tile_cnt = 0;                               // tiles this warp group has consumed so far
        uint32_t done_cnt = 0;                               // items this warp group has finished
        uint32_t pf_cnt = 0;                                 // waits on p_free so far (one per tile but an item's first)
        AtcItem it;
        for (int jj = 0; ok && atc_next(a, jj, it);) {
            const int tile_q0 = it.q0 + w * TQ;
            const int rows_valid = min(TQ, a.seqlen - tile_q0);
            const int qpos = a.pos0 + tile_q0 + row;         // position of this query
            const int n_w = it.n_tiles[w];
            float m_used = -INFINITY, l = 0.f;

            for (int j = 0; j < n_w; ++j, ++tile_cnt) {
                ok = mbar_wait(s_full + w, tile_cnt & 1u, abort_flag);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after_sync();
                float s[TK];
#pragma unroll
                for (int c = 0; c < TK / 32; ++c)
                    tmem_ld_32x32(s_addr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
                tmem_ld_wait();
                if (Cfg::SEPARATE_P) {
                    // the scores are in registers: S_w may take the next tile's scores
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(s_free + w);
                }
                if (j * TK + TK - 1 > a.pos0 + tile_q0) {     // tile holds keys beyond some query of this tile
#pragma unroll
                    for (int i = 0; i < TK; ++i)
                        if (j * TK + i > qpos) s[i] = -INFINITY;
                }
                float mc[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {                 // four independent chains
                    mc[q] = max3f(s[q * 32], s[q * 32 + 1], s[q * 32 + 2]);
#pragma unroll
                    for (int i = 3; i + 1 < 32; i += 2) mc[q] = max3f(mc[q], s[q * 32 + i], s[q * 32 + i + 1]);
                    mc[q] = fmaxf(mc[q], s[q * 32 + 31]);
                }
                const float mx = fmaxf(fmaxf(mc[0], mc[1]), fmaxf(mc[2], mc[3]));
                // raise the maximum in use only when the row's new maximum is far above it
                bool raise = false;
                float f = 1.0f;
                if (j == 0) {
                    m_used = mx;                              // finite: key 0 is visible to every query
                } else {
                    raise = (mx - m_used) * sl2 > RESCALE_LOG2;
                    if (raise) {
                        f = ex2_approx((m_used - mx) * sl2);
                        m_used = mx;
                    }
                }
                if (Cfg::SEPARATE_P && j > 0) {
                    // P_w and (for a rescale) O_w are touched next: the product that read the previous P_w must be
                    // done.  It was issued a whole softmax ago, so this wait succeeds at once.  (The item's first
                    // tile follows the wait for pv_done at the end of the previous item.)
                    ok = mbar_wait(p_free + w, pf_cnt & 1u, abort_flag);
                    ++pf_cnt;
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    tc_fence_after_sync();
                }
                const float neg_ms = -m_used * sl2;
                float sum0 = 0.f, sum1 = 0.f, sum2 = 0.f, sum3 = 0.f;
#pragma unroll
                for (int c = 0; c < TK / 32; ++c) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; i += 2) {
                        float x0 = s[c * 32 + 2 * i], x1 = s[c * 32 + 2 * i + 1];
                        float x2 = s[c * 32 + 2 * i + 2], x3 = s[c * 32 + 2 * i + 3];
                        fma2(x0, x1, sl2, neg_ms);
                        fma2(x2, x3, sl2, neg_ms);
                        x0 = ex2_approx(x0);
                        x1 = ex2_approx(x1);
                        x2 = ex2_approx(x2);
                        x3 = ex2_approx(x3);
                        sum0 += x0;
                        sum1 += x1;
                        sum2 += x2;
                        sum3 += x3;
                        pk[i] = pack_h16x2(x0, x1);
                        pk[i + 1] = pack_h16x2(x2, x3);
                    }
                    tmem_st_32x16(p_addr + c * 16, pk);       // (overwrites scores already consumed when P shares S's columns)
                }
                l = l * f + ((sum0 + sum1) + (sum2 + sum3));
                if (__any_sync(0xFFFFFFFFu, raise)) {
                    // (rare) O_w holds every product issued so far: these scores were committed after the last
                    // one, and a commit covers all that was issued before it.  The next product is not issued
                    // until this warp has released P below.
#pragma unroll 1
                    for (int c = 0; c < HD / 32; ++c) {
                        uint32_t r[32];
                        tmem_ld_32x32(o_addr + c * 32, r);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
                        tmem_st_32x32(o_addr + c * 32, r);
                    }
                }
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_ready + w);
            }
            if (!ok) break;
            if (n_w > 0) {
                ok = mbar_wait(pv_done + w, done_cnt & 1u, abort_flag);   // one arrival per item of this tile slot
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                ++done_cnt;
                tc_fence_after_sync();
                const float inv = 1.f / l;
                const int d = a.n_head * a.head_dim;
                uint16_t *dst = a.out + it.g * a.out_gstride + ((long long)it.b * a.seqlen + tile_q0 + row) * d +
                                it.h * a.head_dim;
#pragma unroll
                for (int c = 0; c < HD / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld_32x32(o_addr + c * 32, r);
                    tmem_ld_wait();
                    if (row < rows_valid) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            if (c * 32 + 8 * i >= a.head_dim) break;
                            uint4 u;
                            u.x = pack_h16x2(__uint_as_float(r[8 * i + 0]) * inv, __uint_as_float(r[8 * i + 1]) * inv);
                            u.y = pack_h16x2(__uint_as_float(r[8 * i + 2]) * inv, __uint_as_float(r[8 * i + 3]) * inv);
                            u.z = pack_h16x2(__uint_as_float(r[8 * i + 4]) * inv, __uint_as_float(r[8 * i + 5]) * inv);
                            u.w = pack_h16x2(__uint_as_float(r[8 * i + 6]) * inv, __uint_as_float(r[8 * i + 7]) * inv);
                            reinterpret_cast<uint4 *>(dst + c * 32)[i] = u;
                        }
                    }
                }
                // the next item's first product may overwrite O_w only after these loads: it waits for
                // this warp group's next p_ready, which comes later in program order
                tc_fence_before_sync();
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
    static DeviceOnce configured;
    if (!configured.done()) {
        int rc = cuda_check(cudaFuncSetAttribute(attn_tc_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 Cfg::SMEM_BYTES), "attention: shared memory opt-in");
        if (rc) return rc;
        configured.set();
    }
    const long long items = (long long)((a.seqlen + 2 * TQ - 1) / (2 * TQ)) * a.n_head * a.batch * a.groups;
    // With more items than SMs, each CTA walks a fixed list of couples of equal total length (atc_next); a plain
    // round-robin list of single items measured slower than one CTA per item (0.38 vs 0.35 ms at 4 x 2048 x 16
    // heads x 128) because the items are so unequal.  KRAKEN_TUNE_ATTN_SCHEDULE = 1 keeps the hardware scheduler.
    const int sms = sm_count() > 0 ? sm_count() : 148;
    const long long couples = (long long)(((a.seqlen + 2 * TQ - 1) / (2 * TQ) + 1) / 2) * a.n_head * a.batch * a.groups;
    AttnTcArgs b = a;
    // The list pays when its rounds fill the machine.  One round (couples <= SMs < items): every couple has an
    // SM of its own and ends together, where the hardware scheduler hands late CTAs the long items (measured at
    // 64 heads x 1024: 29.5 vs 36.1 us).  Several rounds: couples / (SMs x rounds) >= 0.85 (measured: 0.87 gains
    // 7 %, 0.72 loses 3 % against one CTA per item).  With no more items than SMs every item has its own SM and
    // the longest item alone sets the time, which a couple would only lengthen.
    const long long rounds = (couples + sms - 1) / sms;
    b.balanced = items > sms && (rounds == 1 || couples * 100 >= 85LL * sms * rounds) &&
                 tuning(KRAKEN_TUNE_ATTN_SCHEDULE) != 1;
    dim3 grid(static_cast<unsigned>(b.balanced ? (couples < sms ? couples : sms) : items));
    return cuda_check(launch_pdl(attn_tc_kernel<HD>, grid, dim3(ATC_THREADS), Cfg::SMEM_BYTES, stream, tmQ, tmK, tmV, b),
                      "attention: launch");
}

}  // namespace

bool attention_tc_supported(const AttnParams &p) {
    // any head dim that is a multiple of 8 (16-byte rows for TMA) up to 128: the 64- or 128-wide kernel
    // instance runs it with the missing columns zero-filled by the tensor maps
    if (p.head_dim < 16 || p.head_dim > 128 || (p.head_dim & 7)) return false;
    // the cache of one group must be [batch][head][max_pos][head_dim] without gaps
    const int n_kv = p.n_kv_head > 0 ? p.n_kv_head : p.n_head;
    if (p.n_head % n_kv != 0) return false;
    if (p.cache_bstride != (long long)n_kv * p.max_pos * p.head_dim) return false;
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
    const int n_kv = p.n_kv_head > 0 ? p.n_kv_head : p.n_head;
    const uint64_t dims[4] = {(uint64_t)p.head_dim, kv_len, (uint64_t)p.batch * n_kv, (uint64_t)p.groups};
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
    a.n_kv_head = p.n_kv_head > 0 ? p.n_kv_head : p.n_head;
    a.kv_rep = p.n_head / a.n_kv_head;
    a.head_dim = p.head_dim;
    a.out = p.out;
    a.out_gstride = p.out_gstride;
    a.status = d_status;
    return p.head_dim <= 64 ? launch<64>(*tmQ, *tmK, *tmV, a, stream) : launch<128>(*tmQ, *tmK, *tmV, a, stream);
}

}  // namespace kr
