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
    const int n_keys = p.pos_dev ? *p.pos_dev + 1 : p.n_keys;
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
        qf[qh][0] = bf16_lo(u.x) * sl2; qf[qh][1] = bf16_hi(u.x) * sl2; qf[qh][2] = bf16_lo(u.y) * sl2;
        qf[qh][3] = bf16_hi(u.y) * sl2; qf[qh][4] = bf16_lo(u.z) * sl2; qf[qh][5] = bf16_hi(u.z) * sl2;
        qf[qh][6] = bf16_lo(u.w) * sl2; qf[qh][7] = bf16_hi(u.w) * sl2;
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
            kk[u] = active ? *reinterpret_cast<const uint4 *>(gk + off) : make_uint4(0u, 0u, 0u, 0u);
            vv[u] = active ? *reinterpret_cast<const uint4 *>(gv + off) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int qh = 0; qh < QH; ++qh) {
            float s[UNROLL];
            float mx = m[qh];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                float acc = qf[qh][0] * bf16_lo(kk[u].x);
                acc = fmaf(qf[qh][1], bf16_hi(kk[u].x), acc);
                acc = fmaf(qf[qh][2], bf16_lo(kk[u].y), acc);
                acc = fmaf(qf[qh][3], bf16_hi(kk[u].y), acc);
                acc = fmaf(qf[qh][4], bf16_lo(kk[u].z), acc);
                acc = fmaf(qf[qh][5], bf16_hi(kk[u].z), acc);
                acc = fmaf(qf[qh][6], bf16_lo(kk[u].w), acc);
                acc = fmaf(qf[qh][7], bf16_hi(kk[u].w), acc);
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
                    o[qh][0] = fmaf(pu, bf16_lo(vv[u].x), o[qh][0]);
                    o[qh][1] = fmaf(pu, bf16_hi(vv[u].x), o[qh][1]);
                    o[qh][2] = fmaf(pu, bf16_lo(vv[u].y), o[qh][2]);
                    o[qh][3] = fmaf(pu, bf16_hi(vv[u].y), o[qh][3]);
                    o[qh][4] = fmaf(pu, bf16_lo(vv[u].z), o[qh][4]);
                    o[qh][5] = fmaf(pu, bf16_hi(vv[u].z), o[qh][5]);
                    o[qh][6] = fmaf(pu, bf16_lo(vv[u].w), o[qh][6]);
                    o[qh][7] = fmaf(pu, bf16_hi(vv[u].w), o[qh][7]);
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
                    __bfloat16_as_ushort(__float2bfloat16_rn(ot / lt));
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
    p.out[g * p.out_gstride + (long long)b * d + h * HD + e] = __bfloat16_as_ushort(__float2bfloat16_rn(ot / lt));
}

template <int HD>
int launch(const DecodeAttnParams &p, cudaStream_t stream) {
    const int n_kv = p.n_kv_head > 0 ? p.n_kv_head : p.n_head;
    const int rep = p.n_head / n_kv;
    // query heads per CTA: as many of a group as divide it, up to 4 (registers)
    const int qh = rep % 4 == 0 ? 4 : (rep % 2 == 0 ? 2 : 1);
    dim3 grid(p.splits, n_kv * (rep / qh), p.batch * p.groups);
    cudaError_t ce;
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
