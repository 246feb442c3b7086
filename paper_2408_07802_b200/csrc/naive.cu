// Straightforward CUDA-core versions of the GEMM and of attention, one thread (warp) per output.
// They exist for bring-up: with KRAKEN_NAIVE=1 in the environment the model runs on them, which
// separates a scheduling mistake from a tensor-core kernel mistake.  Never used otherwise.
#include <math.h>

#include "epilogue.cuh"
#include "internal.h"

namespace kr {

namespace {


__global__ void gemm_naive_kernel(GemmOperands op, GemmShape s, EpiParams p) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)s.m * s.n_out) return;
    const int row = static_cast<int>(idx / s.n_out), col = static_cast<int>(idx % s.n_out);
    float running = 0.f;
    for (int g = 0; g < s.groups; ++g) {
        const uint16_t *a = static_cast<const uint16_t *>(op.a) + g * op.a_gstride + (long long)row * op.lda;
        const uint16_t *w = static_cast<const uint16_t *>(op.w) + g * op.w_gstride + (long long)col * op.ldw;
        float acc = 0.f;
        for (int k = 0; k < s.k; ++k) acc = fmaf(from_h16(a[k]), from_h16(w[k]), acc);
        if (p.bias) acc += from_h16(p.bias[g * p.bias_gstride + col]);
        switch (p.kind) {
            case KRAKEN_EPI_F32:
                p.out_f32[g * p.out_f32_gstride + (long long)row * p.ld_out_f32 + col] = acc;
                break;
            case KRAKEN_EPI_BF16:
                p.out_bf16[g * p.out_bf16_gstride + (long long)row * p.ld_out_bf16 + col] = to_h16(acc);
                break;
            case KRAKEN_EPI_GELU_BF16:
                p.out_bf16[g * p.out_bf16_gstride + (long long)row * p.ld_out_bf16 + col] =
                    to_h16(gelu_f(acc, p.gelu_tanh));
                break;
            case KRAKEN_EPI_RESID_F32:
            case KRAKEN_EPI_RESID_SUM: {
                const float v = acc + p.resid[g * p.resid_gstride + (long long)row * p.ld_resid + col];
                p.out_f32[g * p.out_f32_gstride + (long long)row * p.ld_out_f32 + col] = v;
                running += v;
                if (p.kind == KRAKEN_EPI_RESID_SUM && g == s.groups - 1) p.sum[(long long)row * p.ld_sum + col] = running;
                break;
            }
            case KRAKEN_EPI_QKV: {
                const int d = p.d_model;
                if (col < d) {
                    p.out_bf16[g * p.out_bf16_gstride + (long long)row * p.ld_out_bf16 + col] = to_h16(acc);
                } else {
                    const int kvd = p.n_kv_head * p.head_dim;
                    const int which = col >= d + kvd, c = col - d - which * kvd;
                    const int head = c / p.head_dim, e = c % p.head_dim;
                    const int b = p.row_seq ? p.row_seq[row] : row / p.seqlen;
                    const int pos = p.row_pos ? p.row_pos[row] : (p.pos0_dev ? p.pos0_dev[b] : p.pos0) + row % p.seqlen;
                    uint16_t *base = (which ? p.v_cache : p.k_cache) + g * p.cache_gstride;
                    base[(((long long)b * p.n_kv_head + head) * p.max_pos + pos) * p.head_dim + e] = to_h16(acc);
                }
                break;
            }
        }
    }
}

// One warp per (group, batch, head, query row): lanes split the head dimension.
__global__ void attention_naive_kernel(AttnParams p) {
    const long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const long long total = (long long)p.groups * p.batch * p.n_head * p.seqlen;
    if (w >= total) return;
    const int t = static_cast<int>(w % p.seqlen);
    const int h = static_cast<int>((w / p.seqlen) % p.n_head);
    const int b = static_cast<int>((w / ((long long)p.seqlen * p.n_head)) % p.batch);
    const int g = static_cast<int>(w / ((long long)p.seqlen * p.n_head * p.batch));
    const int hd = p.head_dim, d = p.n_head * hd;
    const int per = hd / 32;  // 2 or 4 dims per lane
    const uint16_t *q = p.q + g * p.q_gstride + ((long long)b * p.seqlen + t) * d + h * hd;
    const int hk = h / (p.n_head / (p.n_kv_head > 0 ? p.n_kv_head : p.n_head));   // key/value head of this query head
    const uint16_t *kc = p.k_cache + g * p.cache_gstride + b * p.cache_bstride + (long long)hk * p.max_pos * hd;
    const uint16_t *vc = p.v_cache + g * p.cache_gstride + b * p.cache_bstride + (long long)hk * p.max_pos * hd;
    float qv[4], o[4] = {0.f, 0.f, 0.f, 0.f};
    for (int i = 0; i < per; ++i) qv[i] = from_h16(q[lane * per + i]);
    const float scale = rsqrtf(static_cast<float>(hd));
    float m = -INFINITY, l = 0.f;
    for (int j = 0; j <= p.pos0 + t; ++j) {
        float s = 0.f;
        for (int i = 0; i < per; ++i) s += qv[i] * from_h16(kc[(long long)j * hd + lane * per + i]);
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
        s *= scale;
        const float mn = fmaxf(m, s);
        const float corr = __expf(m - mn), e = __expf(s - mn);
        l = l * corr + e;
        for (int i = 0; i < per; ++i) o[i] = o[i] * corr + e * from_h16(vc[(long long)j * hd + lane * per + i]);
        m = mn;
    }
    uint16_t *out = p.out + g * p.out_gstride + ((long long)b * p.seqlen + t) * d + h * hd;
    for (int i = 0; i < per; ++i) out[lane * per + i] = to_h16(o[i] / l);
}

}  // namespace

int launch_gemm_naive(const GemmOperands &op, const GemmShape &s, const EpiParams &epi, cudaStream_t stream) {
    const long long n = (long long)s.m * s.n_out;
    gemm_naive_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, stream>>>(op, s, epi);
    return cudaGetLastError() == cudaSuccess ? KRAKEN_OK : KRAKEN_ECUDA;
}

int launch_attention_naive(const AttnParams &p, cudaStream_t stream) {
    const long long warps = (long long)p.groups * p.batch * p.n_head * p.seqlen;
    attention_naive_kernel<<<static_cast<unsigned>((warps + 7) / 8), 256, 0, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? KRAKEN_OK : KRAKEN_ECUDA;
}

}  // namespace kr
