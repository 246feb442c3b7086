// Decode-step attention: one query row per (branch, sequence, head) against all cached keys.
// Pure HBM streaming of the K/V cache (the dominant bytes of a decode step), so the design is
// about bytes in flight: the keys of one (branch, sequence, head) are split over several CTAs
// (split-KV), every warp issues UNROLL independent 16-byte loads of K and of V per lane before
// it consumes them, rows are read whole and coalesced (8 or 16 lanes per 128/256-byte row),
// scores and the online softmax stay in fp32 registers.  Each split writes an unnormalised
// partial (max, sum, output) to scratch; a second small kernel merges the splits.
#include <math.h>

#include "internal.h"
#include "ptx.cuh"

namespace kr {

namespace {

constexpr int DEC_WARPS = 4;
constexpr int UNROLL = 4;

// QH query heads that share one key/value head (grouped-query attention) are served by one CTA: every
// K and V row is fetched once and used for all of them.  QH = 1 is multi-head attention.
template <int HD, int QH>
__global__ void __launch_bounds__(DEC_WARPS * 32)
attn_decode_kernel(const DecodeAttnParams p) {
    constexpr int LPR = HD / 8;       // lanes that hold one cache row (16 bytes each)
    constexpr int GRP = LPR <= 8 ? 8 : 16;   // lanes set aside per row: the next power of two (the rest idle)
    constexpr int RPW = 32 / GRP;     // rows per warp-wide load
    pdl_wait();
    const int n_kv = p.n_kv_head > 0 ? p.n_kv_head : p.n_head;
    const int rep = p.n_head / n_kv;              // query heads per key/value head
    const int chunks = rep / QH;                  // CTAs per key/value head
    const int split = blockIdx.x;
    const int hk = blockIdx.y / chunks;           // key/value head
    const int h0 = hk * rep + (blockIdx.y % chunks) * QH;   // first query head of this CTA
    const int b = blockIdx.z % p.batch, g = blockIdx.z / p.batch;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane % GRP, rg = lane / GRP;
    const bool active = sub < LPR;
    const int d = p.n_head * HD;

    // keys of this split
    const int n_keys = p.pos_dev ? p.pos_dev[b] + 1 : p.n_keys;
    const int per = (n_keys + p.splits - 1) / p.splits;
    const int k_begin = split * per;
    const int k_end = min(n_keys, k_begin + per);

    const uint16_t *gq = p.q + g * p.q_gstride + (long long)b * d + h0 * HD + (active ? sub : 0) * 8;
    const uint16_t *gk = p.k_cache + g * p.cache_gstride + b * p.cache_bstride + (long long)hk * p.max_pos * HD;
    const uint16_t *gv = p.v_cache + g * p.cache_gstride + b * p.cache_bstride + (long long)hk * p.max_pos * HD;

    // this lane's 8 elements of each query, pre-scaled by log2(e) / sqrt(hd)
    const float sl2 = rsqrtf(static_cast<float>(HD)) * 1.4426950408889634f;
    float qf[QH][8], m[QH], l[QH], o[QH][8];
#pragma unroll
    for (int qh = 0; qh < QH; ++qh) {
        const uint4 u = *reinterpret_cast<const uint4 *>(gq + qh * HD);
        qf[qh][0] = h16_lo(u.x) * sl2; qf[qh][1] = h16_hi(u.x) * sl2; qf[qh][2] = h16_lo(u.y) * sl2;
        qf[qh][3] = h16_hi(u.y) * sl2; qf[qh][4] = h16_lo(u.z) * sl2; qf[qh][5] = h16_hi(u.z) * sl2;
        qf[qh][6] = h16_lo(u.w) * sl2; qf[qh][7] = h16_hi(u.w) * sl2;
        m[qh] = -INFINITY;
        l[qh] = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) o[qh][i] = 0.f;
    }

    // warp w takes row groups w, w + DEC_WARPS, ...; UNROLL groups per iteration
    for (int r0 = k_begin + warp * RPW * UNROLL; r0 < k_end; r0 += DEC_WARPS * RPW * UNROLL) {
        uint4 kk[UNROLL], vv[UNROLL];
        bool valid[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int key = r0 + u * RPW + rg;
            valid[u] = key < k_end;
            const long long off = (long long)(valid[u] ? key : k_begin) * HD + sub * 8;
            kk[u] = active ? __ldcs(reinterpret_cast<const uint4 *>(gk + off)) : make_uint4(0u, 0u, 0u, 0u);
            vv[u] = active ? __ldcs(reinterpret_cast<const uint4 *>(gv + off)) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int qh = 0; qh < QH; ++qh) {
            float s[UNROLL];
            float mx = m[qh];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                float acc = qf[qh][0] * h16_lo(kk[u].x);
                acc = fmaf(qf[qh][1], h16_hi(kk[u].x), acc);
                acc = fmaf(qf[qh][2], h16_lo(kk[u].y), acc);
                acc = fmaf(qf[qh][3], h16_hi(kk[u].y), acc);
                acc = fmaf(qf[qh][4], h16_lo(kk[u].z), acc);
                acc = fmaf(qf[qh][5], h16_hi(kk[u].z), acc);
                acc = fmaf(qf[qh][6], h16_lo(kk[u].w), acc);
                acc = fmaf(qf[qh][7], h16_hi(kk[u].w), acc);
#pragma unroll
                for (int off = 1; off < GRP; off <<= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
                s[u] = valid[u] ? acc : -INFINITY;
                mx = fmaxf(mx, s[u]);
            }
            if (mx > -INFINITY) {  // false only while every key seen by this lane group was out of range
                const float corr = ex2_approx(m[qh] - mx);
                l[qh] *= corr;
#pragma unroll
                for (int i = 0; i < 8; ++i) o[qh][i] *= corr;
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const float pu = ex2_approx(s[u] - mx);
                    l[qh] += pu;
                    o[qh][0] = fmaf(pu, h16_lo(vv[u].x), o[qh][0]);
                    o[qh][1] = fmaf(pu, h16_hi(vv[u].x), o[qh][1]);
                    o[qh][2] = fmaf(pu, h16_lo(vv[u].y), o[qh][2]);
                    o[qh][3] = fmaf(pu, h16_hi(vv[u].y), o[qh][3]);
                    o[qh][4] = fmaf(pu, h16_lo(vv[u].z), o[qh][4]);
                    o[qh][5] = fmaf(pu, h16_hi(vv[u].z), o[qh][5]);
                    o[qh][6] = fmaf(pu, h16_lo(vv[u].w), o[qh][6]);
                    o[qh][7] = fmaf(pu, h16_hi(vv[u].w), o[qh][7]);
                }
                m[qh] = mx;
            }
        }
    }

    pdl_trigger();
    __shared__ float sm_m[QH][DEC_WARPS], sm_l[QH][DEC_WARPS], sm_o[QH][DEC_WARPS][HD];
#pragma unroll
    for (int qh = 0; qh < QH; ++qh) {
        // merge the row groups of the warp (lanes with equal `sub`), then the warps through shared memory
#pragma unroll
        for (int off = GRP; off < 32; off <<= 1) {
            const float m2 = __shfl_xor_sync(0xFFFFFFFFu, m[qh], off);
            const float l2 = __shfl_xor_sync(0xFFFFFFFFu, l[qh], off);
            const float mn = fmaxf(m[qh], m2);
            const float c1 = mn > -INFINITY ? ex2_approx(m[qh] - mn) : 0.f;
            const float c2 = mn > -INFINITY ? ex2_approx(m2 - mn) : 0.f;
            l[qh] = l[qh] * c1 + l2 * c2;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float o2 = __shfl_xor_sync(0xFFFFFFFFu, o[qh][i], off);
                o[qh][i] = o[qh][i] * c1 + o2 * c2;
            }
            m[qh] = mn;
        }
        if (rg == 0 && active) {
#pragma unroll
            for (int i = 0; i < 8; ++i) sm_o[qh][warp][sub * 8 + i] = o[qh][i];
            if (sub == 0) {
                sm_m[qh][warp] = m[qh];
                sm_l[qh][warp] = l[qh];
            }
        }
    }
    __syncthreads();
    if (threadIdx.x < HD) {
        const int e = threadIdx.x;
#pragma unroll
        for (int qh = 0; qh < QH; ++qh) {
            float mn = -INFINITY;
#pragma unroll
            for (int w = 0; w < DEC_WARPS; ++w) mn = fmaxf(mn, sm_m[qh][w]);
            float lt = 0.f, ot = 0.f;
#pragma unroll
            for (int w = 0; w < DEC_WARPS; ++w) {
                const float c = sm_m[qh][w] > -INFINITY ? ex2_approx(sm_m[qh][w] - mn) : 0.f;
                lt += sm_l[qh][w] * c;
                ot += sm_o[qh][w][e] * c;
            }
            const int h = h0 + qh;
            const long long stream = ((long long)blockIdx.z * p.n_head + h);
            if (p.splits == 1) {
                p.out[g * p.out_gstride + (long long)b * d + h * HD + e] =
                    to_h16((ot / lt));
            } else {
                float *part = p.partials + (stream * p.splits + split) * (HD + 2);
                part[2 + e] = ot;
                if (e == 0) {
                    part[0] = mn;
                    part[1] = lt;
                }
            }
        }
    }
}

// Grouped-query decode on the warp-level tensor cores: the query heads that share one key/value head are
// the rows of a 16-row tile, so each cache row fetched from HBM is used for the whole group with one
// m16n8k16 product per 8 keys x 16 head-dim elements instead of one FMA chain and one shuffle tree per head.
//   scores   S[head, key] = sum_e Q[head, e] K[key, e]: a lane loads 16 bytes (8 consecutive e) of one key
//            and feeds them to two products; Q is held in registers with the same placement of e in the
//            k slots, which is all a dot product needs (the order of e does not matter);
//   output   O[head, e] += sum_key P[head, key] V[key, e]: P comes straight from the score accumulators
//            (the accumulator layout of two 8-key blocks is the A layout of one 16-key product); a lane
//            loads 16 bytes (8 consecutive e) of four keys and pairs elements of neighbouring keys with a
//            byte permute, so product j of a 64-column half yields columns 8 n + j: every lane ends up
//            with runs of 8 consecutive output columns.
// One CTA per (group, sequence, key/value head, split); its 4 warps take 16-key blocks in turn, each with
// its own running maximum and sum per head, merged through shared memory at the end.
__device__ __forceinline__ void mma16816_dec(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32." KRAKEN_MMA_T "." KRAKEN_MMA_T ".f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t u4_elem(const uint4 &v, int i) { return i == 0 ? v.x : (i == 1 ? v.y : (i == 2 ? v.z : v.w)); }

constexpr int GQA_ROWS = 16;   // query heads per key/value head served by one tile (rows beyond the group are zero)

template <int HD>
__global__ void __launch_bounds__(DEC_WARPS * 32)
attn_decode_gqa_kernel(const DecodeAttnParams p) {
    constexpr int CH = HD / 32;   // 32-element chunks of the head dim (scores)
    constexpr int HF = HD / 64;   // 64-column halves of the head dim (output)
    pdl_wait();
    const int n_kv = p.n_kv_head;
    const int rep = p.n_head / n_kv;              // query heads per key/value head, <= GQA_ROWS
    const int split = blockIdx.x, hk = blockIdx.y;
    const int h0 = hk * rep;
    const int b = blockIdx.z % p.batch, g = blockIdx.z / p.batch;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kq = lane & 3, nq = lane >> 2;
    const int d = p.n_head * HD;

    const int n_keys = p.pos_dev ? p.pos_dev[b] + 1 : p.n_keys;
    const int per = (n_keys + p.splits - 1) / p.splits;
    const int k_begin = split * per;
    const int k_end = min(n_keys, k_begin + per);

    const uint16_t *gq = p.q + g * p.q_gstride + (long long)b * d + h0 * HD;
    const uint16_t *gk = p.k_cache + g * p.cache_gstride + b * p.cache_bstride + (long long)hk * p.max_pos * HD;
    const uint16_t *gv = p.v_cache + g * p.cache_gstride + b * p.cache_bstride + (long long)hk * p.max_pos * HD;
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);

    // Q: rows nq and nq + 8 of the tile, this lane's 8 elements of every 32-element chunk
    uint4 qa[CH][2];
#pragma unroll
    for (int c = 0; c < CH; ++c)
#pragma unroll
        for (int hl = 0; hl < 2; ++hl) {
            const int row = hl * 8 + nq;
            qa[c][hl] = row < rep ? *reinterpret_cast<const uint4 *>(gq + row * HD + c * 32 + kq * 8) : zero;
        }
    const float sl2 = rsqrtf(static_cast<float>(HD)) * 1.4426950408889634f;
    float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
    float o[HF * 8][4];
#pragma unroll
    for (int j = 0; j < HF * 8; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;

    for (int r0 = k_begin + warp * 16; r0 < k_end; r0 += DEC_WARPS * 16) {
        // K: two blocks of 8 keys, key = block * 8 + nq; V: keys kq*2, kq*2+1 of both blocks, columns nq*8..+7
        uint4 kk[2][CH], vv[4][HF];
#pragma unroll
        for (int kb = 0; kb < 2; ++kb) {
            const int key = r0 + kb * 8 + nq;
#pragma unroll
            for (int c = 0; c < CH; ++c)
                kk[kb][c] = key < k_end ? __ldcs(reinterpret_cast<const uint4 *>(gk + (long long)key * HD + c * 32 + kq * 8)) : zero;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int key = r0 + (i >> 1) * 8 + kq * 2 + (i & 1);
#pragma unroll
            for (int hf = 0; hf < HF; ++hf)
                vv[i][hf] = key < k_end ? __ldcs(reinterpret_cast<const uint4 *>(gv + (long long)key * HD + hf * 64 + nq * 8)) : zero;
        }
        float s[2][4];
#pragma unroll
        for (int kb = 0; kb < 2; ++kb) {
            s[kb][0] = s[kb][1] = s[kb][2] = s[kb][3] = 0.f;
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                mma16816_dec(s[kb], qa[c][0].x, qa[c][1].x, qa[c][0].y, qa[c][1].y, kk[kb][c].x, kk[kb][c].y);
                mma16816_dec(s[kb], qa[c][0].z, qa[c][1].z, qa[c][0].w, qa[c][1].w, kk[kb][c].z, kk[kb][c].w);
            }
            // columns of this lane: keys r0 + kb*8 + kq*2 + {0, 1}
            const int key0 = r0 + kb * 8 + kq * 2;
            s[kb][0] = key0 < k_end ? s[kb][0] * sl2 : -INFINITY;
            s[kb][2] = key0 < k_end ? s[kb][2] * sl2 : -INFINITY;
            s[kb][1] = key0 + 1 < k_end ? s[kb][1] * sl2 : -INFINITY;
            s[kb][3] = key0 + 1 < k_end ? s[kb][3] * sl2 : -INFINITY;
        }
        uint32_t pa[4];   // P as the A operand of the 16-key product
#pragma unroll
        for (int hl = 0; hl < 2; ++hl) {
            float mx = fmaxf(fmaxf(s[0][2 * hl], s[0][2 * hl + 1]), fmaxf(s[1][2 * hl], s[1][2 * hl + 1]));
            mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 2));
            mx = fmaxf(mx, m[hl]);                 // finite: key r0 is in range and belongs to this quad's columns
            const float corr = ex2_approx(m[hl] - mx);
            m[hl] = mx;
            const float p00 = ex2_approx(s[0][2 * hl] - mx), p01 = ex2_approx(s[0][2 * hl + 1] - mx);
            const float p10 = ex2_approx(s[1][2 * hl] - mx), p11 = ex2_approx(s[1][2 * hl + 1] - mx);
            l[hl] = l[hl] * corr + ((p00 + p01) + (p10 + p11));    // this lane's columns; summed over the quad at the end
            pa[hl] = pack_h16x2(p00, p01);
            pa[2 + hl] = pack_h16x2(p10, p11);
#pragma unroll
            for (int j = 0; j < HF * 8; ++j) {
                o[j][2 * hl] *= corr;
                o[j][2 * hl + 1] *= corr;
            }
        }
#pragma unroll
        for (int hf = 0; hf < HF; ++hf)
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                // element j of the 8 columns each key row piece holds: low half from the even key, high half from the odd
                const uint32_t sel = (j & 1) ? 0x7632u : 0x5410u;
                const uint32_t b0 = __byte_perm(u4_elem(vv[0][hf], j >> 1), u4_elem(vv[1][hf], j >> 1), sel);
                const uint32_t b1 = __byte_perm(u4_elem(vv[2][hf], j >> 1), u4_elem(vv[3][hf], j >> 1), sel);
                mma16816_dec(o[hf * 8 + j], pa[0], pa[1], pa[2], pa[3], b0, b1);
            }
    }

    pdl_trigger();
    // row sums over the quad; then the 4 warps through shared memory
#pragma unroll
    for (int hl = 0; hl < 2; ++hl) {
        l[hl] += __shfl_xor_sync(0xFFFFFFFFu, l[hl], 1);
        l[hl] += __shfl_xor_sync(0xFFFFFFFFu, l[hl], 2);
    }
    __shared__ float sm_m[DEC_WARPS][GQA_ROWS], sm_l[DEC_WARPS][GQA_ROWS];
    __shared__ float sm_o[DEC_WARPS][GQA_ROWS][HD];
#pragma unroll
    for (int hl = 0; hl < 2; ++hl) {
        const int row = hl * 8 + nq;
        if (row < rep) {
            if (kq == 0) {
                sm_m[warp][row] = m[hl];
                sm_l[warp][row] = l[hl];
            }
            // accumulator (hf, j), element 2 hl + e: column hf*64 + (kq*2 + e)*8 + j
#pragma unroll
            for (int hf = 0; hf < HF; ++hf)
#pragma unroll
                for (int e = 0; e < 2; ++e)
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        sm_o[warp][row][hf * 64 + (kq * 2 + e) * 8 + j] = o[hf * 8 + j][2 * hl + e];
        }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < rep * HD; idx += DEC_WARPS * 32) {
        const int row = idx / HD, e = idx % HD;
        float mn = -INFINITY;
#pragma unroll
        for (int w = 0; w < DEC_WARPS; ++w) mn = fmaxf(mn, sm_m[w][row]);
        float lt = 0.f, ot = 0.f;
#pragma unroll
        for (int w = 0; w < DEC_WARPS; ++w) {
            const float c = sm_m[w][row] > -INFINITY ? ex2_approx(sm_m[w][row] - mn) : 0.f;
            lt += sm_l[w][row] * c;
            ot += sm_o[w][row][e] * c;
        }
        const int h = h0 + row;
        const long long stream = ((long long)blockIdx.z * p.n_head + h);
        if (p.splits == 1) {
            p.out[g * p.out_gstride + (long long)b * d + h * HD + e] = to_h16((ot / lt));
        } else {
            float *part = p.partials + (stream * p.splits + split) * (HD + 2);
            part[2 + e] = ot;
            if (e == 0) {
                part[0] = mn;
                part[1] = lt;
            }
        }
    }
}

// out = sum_s o_s 2^(m_s - m) / sum_s l_s 2^(m_s - m)
template <int HD>
__global__ void __launch_bounds__(HD) attn_decode_merge_kernel(const DecodeAttnParams p) {
    pdl_wait();
    pdl_trigger();
    const int h = blockIdx.x;
    const int b = blockIdx.y % p.batch, g = blockIdx.y / p.batch;
    const int e = threadIdx.x;
    const long long stream = ((long long)blockIdx.y * p.n_head + h);
    const float *part = p.partials + stream * p.splits * (HD + 2);
    float mn = -INFINITY;
    for (int s = 0; s < p.splits; ++s) mn = fmaxf(mn, part[s * (HD + 2)]);
    float lt = 0.f, ot = 0.f;
    for (int s = 0; s < p.splits; ++s) {
        const float ms = part[s * (HD + 2)];
        const float c = ms > -INFINITY ? ex2_approx(ms - mn) : 0.f;
        lt += part[s * (HD + 2) + 1] * c;
        ot += part[s * (HD + 2) + 2 + e] * c;
    }
    const int d = p.n_head * HD;
    p.out[g * p.out_gstride + (long long)b * d + h * HD + e] = to_h16((ot / lt));
}

template <int HD>
int launch(const DecodeAttnParams &p, cudaStream_t stream) {
    const int n_kv = p.n_kv_head > 0 ? p.n_kv_head : p.n_head;
    const int rep = p.n_head / n_kv;
    // query heads per CTA: as many of a group as divide it, up to 4 (registers)
    const int qh = rep % 4 == 0 ? 4 : (rep % 2 == 0 ? 2 : 1);
    dim3 grid(p.splits, n_kv * (rep / qh), p.batch * p.groups);
    cudaError_t ce;
    if constexpr (HD == 64 || HD == 128) {
        if (decode_gqa_tile(p.n_head, n_kv)) {
            DecodeAttnParams q = p;
            q.n_kv_head = n_kv;
            ce = launch_pdl(attn_decode_gqa_kernel<HD>, dim3(p.splits, n_kv, p.batch * p.groups), dim3(DEC_WARPS * 32), 0,
                            stream, q);
            int rc = cuda_check(ce, "grouped decode attention: launch");
            if (rc) return rc;
            if (p.splits > 1) {
                dim3 g2(p.n_head, p.batch * p.groups);
                rc = cuda_check(launch_pdl(attn_decode_merge_kernel<HD>, g2, dim3(HD), 0, stream, p),
                                "decode attention merge: launch");
            }
            return rc;
        }
    }
    if (qh == 4) ce = launch_pdl(attn_decode_kernel<HD, 4>, grid, dim3(DEC_WARPS * 32), 0, stream, p);
    else if (qh == 2) ce = launch_pdl(attn_decode_kernel<HD, 2>, grid, dim3(DEC_WARPS * 32), 0, stream, p);
    else ce = launch_pdl(attn_decode_kernel<HD, 1>, grid, dim3(DEC_WARPS * 32), 0, stream, p);
    int rc = cuda_check(ce, "decode attention: launch");
    if (rc) return rc;
    if (p.splits > 1) {
        dim3 g2(p.n_head, p.batch * p.groups);
        rc = cuda_check(launch_pdl(attn_decode_merge_kernel<HD>, g2, dim3(HD), 0, stream, p),
                        "decode attention merge: launch");
    }
    return rc;
}

}  // namespace

// whether the tensor-core tile kernel serves this grouping (2 .. 16 query heads per key/value head)
bool decode_gqa_tile(int n_head, int n_kv_head) {
    if (n_kv_head < 1 || n_head % n_kv_head != 0) return false;
    const int rep = n_head / n_kv_head;
    return rep >= 2 && rep <= GQA_ROWS;
}

int decode_attention_splits(int groups, int batch, int n_head, int n_keys) {
    const long long streams = (long long)groups * batch * n_head;
    const int sms = sm_count() > 0 ? sm_count() : 148;
    const long long want = 6LL * sms;  // CTAs to aim for
    long long s = (want + streams - 1) / streams;
    const long long by_len = (n_keys + 127) / 128;  // at least 128 keys per split
    if (s > by_len) s = by_len;
    if (s > DECODE_MAX_SPLITS) s = DECODE_MAX_SPLITS;
    if (s < 1) s = 1;
    return static_cast<int>(s);
}

size_t decode_attention_partial_bytes(int groups, int batch, int n_head, int head_dim, int splits) {
    return (size_t)groups * batch * n_head * splits * (head_dim + 2) * sizeof(float);
}

int launch_attention_decode(const DecodeAttnParams &p, cudaStream_t stream) {
    if (!p.q || !p.k_cache || !p.v_cache || !p.out || p.groups < 1 || p.batch < 1 || p.n_head < 1 || p.n_keys < 1 ||
        p.n_keys > p.max_pos || p.splits < 1 || p.splits > DECODE_MAX_SPLITS || (p.splits > 1 && !p.partials))
        return KRAKEN_EINVAL;
    if (p.n_kv_head < 0 || (p.n_kv_head > 0 && p.n_head % p.n_kv_head != 0)) return KRAKEN_EINVAL;
    switch (p.head_dim) {   // 64 and 128, and the head dims of the paper's engine shapes (Table 3)
        case 64: return launch<64>(p, stream);
        case 72: return launch<72>(p, stream);
        case 96: return launch<96>(p, stream);
        case 104: return launch<104>(p, stream);
        case 128: return launch<128>(p, stream);
        default: return KRAKEN_EUNSUPPORTED;
    }
}

}  // namespace kr
