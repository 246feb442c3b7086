// Weight-streaming GEMM for a handful of rows (decode steps and the last-position tail):
// C_g[M, Nout] = A_g[M, K] . W_g[Nout, K]^T with M <= 32.  Every weight byte is read exactly once,
// so the kernel is bound by HBM and shaped for bytes in flight, not for the tensor pipe:
//   - one CTA per strip of 8 output columns of one group, 4 or 8 warps splitting K;
//   - every lane streams 16-byte pieces of a weight row (4 lanes cover 64 contiguous bytes of each
//     of 8 rows) and the matching 16-byte pieces of the activation rows (L1/L2 resident);
//   - products run on m16n8k16 warp MMAs with the K slots permuted identically for both operands,
//     which is what lets plain 16-byte loads feed the fragments without a shuffle;
//   - the 8 partial sums of an output are added in a fixed order (deterministic), then the fused
//     epilogue runs per element.
#include "epilogue.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace kr {

namespace {

constexpr int SK_COLS = 8;
constexpr int SK_UNROLL = 8;

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32." KRAKEN_MMA_T "." KRAKEN_MMA_T ".f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}


// Epilogue of one output element (same semantics as the tile epilogue of the tensor-core GEMM,
// except KRAKEN_EPI_RESID_SUM, which this kernel does not take: callers sum small tensors elsewhere).
__device__ __forceinline__ void epilogue_elem(const EpiParams &p, int g, int row, int col, float acc) {
    if (p.bias) acc += from_h16(p.bias[g * p.bias_gstride + col]);
    switch (p.kind) {
        case KRAKEN_EPI_F32:
            p.out_f32[g * p.out_f32_gstride + (long long)row * p.ld_out_f32 + col] = acc;
            break;
        case KRAKEN_EPI_BF16:
            p.out_bf16[g * p.out_bf16_gstride + (long long)row * p.ld_out_bf16 + col] = to_h16(acc);
            break;
        case KRAKEN_EPI_GELU_BF16:
            p.out_bf16[g * p.out_bf16_gstride + (long long)row * p.ld_out_bf16 + col] = to_h16(gelu_f(acc, p.gelu_tanh));
            break;
        case KRAKEN_EPI_RESID_F32:
            p.out_f32[g * p.out_f32_gstride + (long long)row * p.ld_out_f32 + col] =
                acc + p.resid[g * p.resid_gstride + (long long)row * p.ld_resid + col];
            break;
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
        default:
            break;
    }
}

template <int MB, int SK_WARPS>  // 16-row blocks of A (1 or 2); warps splitting K
__global__ void __launch_bounds__(SK_WARPS * 32)
gemm_skinny_kernel(const GemmOperands op, const GemmShape s, const EpiParams epi) {
    pdl_wait();
    const int g = blockIdx.y;
    const int n0 = blockIdx.x * SK_COLS;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nn = lane >> 2, kq = lane & 3;

    // K range of this warp, in chunks of 32
    const int chunks = (s.k + 31) / 32;
    const int per = (chunks + SK_WARPS - 1) / SK_WARPS;
    const int c_begin = warp * per, c_end = min(chunks, c_begin + per);

    const uint16_t *A = static_cast<const uint16_t *>(op.a) + g * op.a_gstride;
    const bool n_ok = n0 + nn < s.n_out;
    const uint16_t *wrow = static_cast<const uint16_t *>(op.w) + g * op.w_gstride + (long long)(n_ok ? n0 + nn : 0) * op.ldw;
    const uint16_t *arow[MB][2];
    bool a_ok[MB][2];
#pragma unroll
    for (int mb = 0; mb < MB; ++mb)
#pragma unroll
        for (int hlf = 0; hlf < 2; ++hlf) {
            const int r = mb * 16 + hlf * 8 + nn;
            a_ok[mb][hlf] = r < s.m;
            arow[mb][hlf] = A + (long long)(a_ok[mb][hlf] ? r : 0) * op.lda;
        }

    float acc[MB][4];
#pragma unroll
    for (int mb = 0; mb < MB; ++mb) acc[mb][0] = acc[mb][1] = acc[mb][2] = acc[mb][3] = 0.f;
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);

    for (int c0 = c_begin; c0 < c_end; c0 += SK_UNROLL) {
        // the weight pieces of the whole batch go in flight first (they come from DRAM); the activation
        // pieces are fetched chunk by chunk right before use (they sit in L1/L2), which keeps the
        // register count low enough for eight CTAs per SM
        uint4 wv[SK_UNROLL];
#pragma unroll
        for (int u = 0; u < SK_UNROLL; ++u) {
            const int k = (c0 + u) * 32 + kq * 8;
            const bool k_ok = (c0 + u) < c_end && k < s.k;
            wv[u] = (k_ok && n_ok) ? __ldcs(reinterpret_cast<const uint4 *>(wrow + k)) : zero;
        }
#pragma unroll
        for (int u = 0; u < SK_UNROLL; ++u) {
            const int k = (c0 + u) * 32 + kq * 8;
            const bool k_ok = (c0 + u) < c_end && k < s.k;
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) {
                const uint4 a0 = (k_ok && a_ok[mb][0]) ? *reinterpret_cast<const uint4 *>(arow[mb][0] + k) : zero;
                const uint4 a1 = (k_ok && a_ok[mb][1]) ? *reinterpret_cast<const uint4 *>(arow[mb][1] + k) : zero;
                mma16816(acc[mb], a0.x, a1.x, a0.y, a1.y, wv[u].x, wv[u].y);
                mma16816(acc[mb], a0.z, a1.z, a0.w, a1.w, wv[u].z, wv[u].w);
            }
        }
    }

    pdl_trigger();
    // cross-warp reduction in a fixed order
    __shared__ float part[SK_WARPS][MB * 16][SK_COLS];
#pragma unroll
    for (int mb = 0; mb < MB; ++mb) {
        part[warp][mb * 16 + nn][kq * 2] = acc[mb][0];
        part[warp][mb * 16 + nn][kq * 2 + 1] = acc[mb][1];
        part[warp][mb * 16 + 8 + nn][kq * 2] = acc[mb][2];
        part[warp][mb * 16 + 8 + nn][kq * 2 + 1] = acc[mb][3];
    }
    __syncthreads();
    for (int e = threadIdx.x; e < MB * 16 * SK_COLS; e += SK_WARPS * 32) {
        const int row = e / SK_COLS, col = n0 + e % SK_COLS;
        if (row < s.m && col < s.n_out) {
            float v = 0.f;
#pragma unroll
            for (int w = 0; w < SK_WARPS; ++w) v += part[w][row][e % SK_COLS];
            epilogue_elem(epi, g, row, col, v);
        }
    }
}

}  // namespace

int launch_gemm_skinny(const GemmOperands &op, const GemmShape &s, const EpiParams &epi, cudaStream_t stream) {
    if (s.groups < 1 || s.m < 1 || s.m > 32 || s.n_out < 1 || s.k < 8 || (s.k & 7)) return KRAKEN_EINVAL;
    if (epi.kind == KRAKEN_EPI_RESID_SUM) return KRAKEN_EUNSUPPORTED;
    if ((op.lda & 7) || (op.ldw & 7) || (reinterpret_cast<uintptr_t>(op.a) & 15) ||
        (reinterpret_cast<uintptr_t>(op.w) & 15) || (op.a_gstride & 7) || (op.w_gstride & 7))
        return KRAKEN_EUNSUPPORTED;
    dim3 grid((s.n_out + SK_COLS - 1) / SK_COLS, s.groups);
    // K is split over the warps of a CTA so that each warp still streams a few hundred bytes per lane
    const bool wide_k = s.k > 2048;
    cudaError_t ce;
    if (s.m <= 16) {
        ce = wide_k ? launch_pdl(gemm_skinny_kernel<1, 8>, grid, dim3(256), 0, stream, op, s, epi)
                    : launch_pdl(gemm_skinny_kernel<1, 4>, grid, dim3(128), 0, stream, op, s, epi);
    } else {
        ce = wide_k ? launch_pdl(gemm_skinny_kernel<2, 8>, grid, dim3(256), 0, stream, op, s, epi)
                    : launch_pdl(gemm_skinny_kernel<2, 4>, grid, dim3(128), 0, stream, op, s, epi);
    }
    return cuda_check(ce, "skinny gemm: launch");
}

}  // namespace kr
