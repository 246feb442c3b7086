// Causal multi-head attention for prefill: softmax(q k^T / sqrt(hd)) v per (branch, sequence, head),
// streaming over K/V tiles of the cache with an online softmax (no l x l matrix is ever stored).
//
// One CTA = 64 query rows of one head (4 warps x 16 rows); K/V tiles of 64 keys are staged in
// shared memory with cp.async (double buffered, 16-byte chunks XOR-swizzled against bank
// conflicts); both products run on the tensor cores with warp-level m16n8k16 MMAs; the
// probabilities never leave registers.  Query tiles are launched longest first.
#include <math.h>

#include "internal.h"
#include "ptx.cuh"

namespace kr {

namespace {

constexpr int ABM = 64;  // query rows per CTA
constexpr int ABN = 64;  // keys per tile

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src, bool valid) {
    const int sz = valid ? 16 : 0;  // size 0: destination is zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32." KRAKEN_MMA_T "." KRAKEN_MMA_T ".f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// element offset of (row, 16-byte chunk) in a [rows][HD] bf16 tile
template <int HD>
__device__ __forceinline__ int swz(int row, int chunk) {
    return row * HD + ((chunk ^ (row & 7)) << 3);
}

template <int HD>
__global__ void __launch_bounds__(128) attn_prefill_kernel(const AttnParams p) {
    constexpr int CH = HD / 8;    // 16-byte chunks per row
    constexpr int KS = HD / 16;   // k-steps of q.k^T; also pairs of 8-wide output column tiles
    extern __shared__ __align__(128) uint16_t smem_attn[];
    uint16_t *sQ = smem_attn;
    uint16_t *sK = sQ + ABM * HD;       // [2][ABN][HD]
    uint16_t *sV = sK + 2 * ABN * HD;   // [2][ABN][HD]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int mt = gridDim.x - 1 - blockIdx.x;  // longest rows first
    const int h = blockIdx.y;
    const int b = blockIdx.z % p.batch, g = blockIdx.z / p.batch;
    const int d = p.n_head * HD;
    const int q0 = mt * ABM;
    const int rows_valid = min(ABM, p.seqlen - q0);
    const int kv_len = p.pos0 + p.seqlen;                 // keys that hold data
    const int n_keys = p.pos0 + q0 + rows_valid;          // keys visible to the last row of this tile
    const int n_tiles = (n_keys + ABN - 1) / ABN;

    const uint16_t *gq = p.q + g * p.q_gstride + ((long long)b * p.seqlen + q0) * d + h * HD;
    const uint16_t *gk = p.k_cache + g * p.cache_gstride + b * p.cache_bstride + (long long)h * p.max_pos * HD;
    const uint16_t *gv = p.v_cache + g * p.cache_gstride + b * p.cache_bstride + (long long)h * p.max_pos * HD;

    auto load_kv = [&](int tile, int buf) {
        for (int c = tid; c < ABN * CH; c += 128) {
            const int r = c / CH, ch = c % CH;
            const int key = tile * ABN + r;
            const bool valid = key < kv_len;
            const long long off = (long long)(valid ? key : 0) * HD + ch * 8;
            cp_async_16(smem_u32(sK + buf * ABN * HD + swz<HD>(r, ch)), gk + off, valid);
            cp_async_16(smem_u32(sV + buf * ABN * HD + swz<HD>(r, ch)), gv + off, valid);
        }
    };
    for (int c = tid; c < ABM * CH; c += 128) {
        const int r = c / CH, ch = c % CH;
        const bool valid = r < rows_valid;
        cp_async_16(smem_u32(sQ + swz<HD>(r, ch)), gq + (long long)(valid ? r : 0) * d + ch * 8, valid);
    }
    load_kv(0, 0);
    cp_async_commit();

    const float sl2 = rsqrtf(static_cast<float>(HD)) * 1.4426950408889634f;  // scale * log2(e)
    uint32_t qf[KS][4];
    float acc[HD / 8][4];
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
    float m_i[2] = {-INFINITY, -INFINITY}, l_i[2] = {0.f, 0.f};
    const int qpos0 = p.pos0 + q0 + warp * 16 + (lane >> 2);  // position of this thread's first row

    for (int j = 0; j < n_tiles; ++j) {
        const int buf = j & 1;
        if (j + 1 < n_tiles) load_kv(j + 1, buf ^ 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        if (j == 0) {
#pragma unroll
            for (int ks = 0; ks < KS; ++ks)
                ldmatrix_x4(qf[ks], smem_u32(sQ + swz<HD>(warp * 16 + (lane & 15), ks * 2 + (lane >> 4))));
        }
        const uint16_t *tK = sK + buf * ABN * HD;
        const uint16_t *tV = sV + buf * ABN * HD;

        float s[ABN / 8][4];
#pragma unroll
        for (int i = 0; i < ABN / 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
            for (int np = 0; np < ABN / 16; ++np) {
                uint32_t kf[4];
                ldmatrix_x4(kf, smem_u32(tK + swz<HD>(np * 16 + (lane & 7) + ((lane >> 4) << 3),
                                                      ks * 2 + ((lane >> 3) & 1))));
                mma_bf16_16816(s[2 * np], qf[ks], kf[0], kf[1]);
                mma_bf16_16816(s[2 * np + 1], qf[ks], kf[2], kf[3]);
            }
        }
        // causal mask: key position > query position is excluded
        if (j * ABN + ABN - 1 > p.pos0 + q0 + warp * 16) {
#pragma unroll
            for (int nt = 0; nt < ABN / 8; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int key = j * ABN + nt * 8 + ((lane & 3) << 1) + (e & 1);
                    const int qpos = qpos0 + ((e >> 1) << 3);
                    if (key > qpos) s[nt][e] = -INFINITY;
                }
        }
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < ABN / 8; ++nt) {
            mx[0] = fmaxf(mx[0], fmaxf(s[nt][0], s[nt][1]));
            mx[1] = fmaxf(mx[1], fmaxf(s[nt][2], s[nt][3]));
        }
        float corr[2], mscaled[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xFFFFFFFFu, mx[r], 1));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xFFFFFFFFu, mx[r], 2));
            const float m_new = fmaxf(m_i[r], mx[r]);  // finite: key 0 is visible to every row
            corr[r] = ex2_approx((m_i[r] - m_new) * sl2);
            m_i[r] = m_new;
            mscaled[r] = m_new * sl2;
        }
        float rs[2] = {0.f, 0.f};
#pragma unroll
        for (int nt = 0; nt < ABN / 8; ++nt) {
            s[nt][0] = ex2_approx(s[nt][0] * sl2 - mscaled[0]);
            s[nt][1] = ex2_approx(s[nt][1] * sl2 - mscaled[0]);
            s[nt][2] = ex2_approx(s[nt][2] * sl2 - mscaled[1]);
            s[nt][3] = ex2_approx(s[nt][3] * sl2 - mscaled[1]);
            rs[0] += s[nt][0] + s[nt][1];
            rs[1] += s[nt][2] + s[nt][3];
        }
        l_i[0] = l_i[0] * corr[0] + rs[0];
        l_i[1] = l_i[1] * corr[1] + rs[1];
#pragma unroll
        for (int i = 0; i < HD / 8; ++i) {
            acc[i][0] *= corr[0];
            acc[i][1] *= corr[0];
            acc[i][2] *= corr[1];
            acc[i][3] *= corr[1];
        }
#pragma unroll
        for (int kk = 0; kk < ABN / 16; ++kk) {
            uint32_t pf[4];
            pf[0] = pack_h16x2(s[2 * kk][0], s[2 * kk][1]);
            pf[1] = pack_h16x2(s[2 * kk][2], s[2 * kk][3]);
            pf[2] = pack_h16x2(s[2 * kk + 1][0], s[2 * kk + 1][1]);
            pf[3] = pack_h16x2(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
            for (int dp = 0; dp < KS; ++dp) {
                uint32_t vf[4];
                ldmatrix_x4_trans(vf, smem_u32(tV + swz<HD>(kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3),
                                                            dp * 2 + (lane >> 4))));
                mma_bf16_16816(acc[2 * dp], pf, vf[0], vf[1]);
                mma_bf16_16816(acc[2 * dp + 1], pf, vf[2], vf[3]);
            }
        }
        __syncthreads();  // everyone is done with this buffer before it is refilled
    }
    cp_async_wait<0>();

#pragma unroll
    for (int r = 0; r < 2; ++r) {
        l_i[r] += __shfl_xor_sync(0xFFFFFFFFu, l_i[r], 1);
        l_i[r] += __shfl_xor_sync(0xFFFFFFFFu, l_i[r], 2);
    }
    const float inv0 = 1.f / l_i[0], inv1 = 1.f / l_i[1];
    const int r0 = warp * 16 + (lane >> 2), r1 = r0 + 8;
    uint16_t *go = p.out + g * p.out_gstride + ((long long)b * p.seqlen + q0) * d + h * HD;
#pragma unroll
    for (int nt = 0; nt < HD / 8; ++nt) {
        const int col = nt * 8 + ((lane & 3) << 1);
        if (r0 < rows_valid)
            *reinterpret_cast<uint32_t *>(go + (long long)r0 * d + col) = pack_h16x2(acc[nt][0] * inv0, acc[nt][1] * inv0);
        if (r1 < rows_valid)
            *reinterpret_cast<uint32_t *>(go + (long long)r1 * d + col) = pack_h16x2(acc[nt][2] * inv1, acc[nt][3] * inv1);
    }
}

template <int HD>
int launch(const AttnParams &p, cudaStream_t stream) {
    constexpr int smem = (ABM + 4 * ABN) * HD * 2;
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(attn_prefill_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) !=
            cudaSuccess)
            return KRAKEN_ECUDA;
        configured = true;
    }
    dim3 grid((p.seqlen + ABM - 1) / ABM, p.n_head, p.batch * p.groups);
    attn_prefill_kernel<HD><<<grid, 128, smem, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? KRAKEN_OK : KRAKEN_ECUDA;
}

}  // namespace

int launch_attention_prefill(const AttnParams &p, cudaStream_t stream) {
    if (!p.q || !p.k_cache || !p.v_cache || !p.out || p.groups < 1 || p.batch < 1 || p.seqlen < 1 || p.pos0 < 0 ||
        p.n_head < 1 || p.pos0 + p.seqlen > p.max_pos)
        return KRAKEN_EINVAL;
    if (p.head_dim == 64) return launch<64>(p, stream);
    if (p.head_dim == 128) return launch<128>(p, stream);
    return KRAKEN_EUNSUPPORTED;
}

}  // namespace kr
