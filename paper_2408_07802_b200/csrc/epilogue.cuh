// Fused GEMM epilogues (bias, GELU, residual add, cross-branch sum, K/V scatter into the cache).
#pragma once
#include "internal.h"
#include "ptx.cuh"

namespace kr {

// erf by the rational-times-Gaussian form 1 - (a1 t + ... + a5 t^5) exp(-z^2), t = 1 / (1 + p z)
// (Abramowitz & Stegun 7.1.26, |error| <= 1.5e-7): branch-free, two special-function-unit ops.
__device__ __forceinline__ float erf_as(float z) {
    const float az = fabsf(z);
    const float t = rcp_approx(fmaf(0.3275911f, az, 1.0f));
    float poly = fmaf(1.061405429f, t, -1.453152027f);
    poly = fmaf(poly, t, 1.421413741f);
    poly = fmaf(poly, t, -0.284496736f);
    poly = fmaf(poly, t, 0.254829592f);
    poly *= t;
    const float e = ex2_approx(-1.4426950408889634f * az * az);
    return copysignf(fmaf(-poly, e, 1.0f), z);
}

__device__ __forceinline__ float gelu_f(float x, int tanh_form) {
    if (tanh_form) {
        const float c = 0.7978845608028654f;
        return 0.5f * x * (1.0f + tanhf(c * (x + 0.044715f * x * x * x)));
    }
    return 0.5f * x * (1.0f + erf_as(x * 0.7071067811865476f));
}

// GELU (erf form) of two values at once on the packed fp32 pipe; same formula as erf_as.
__device__ __forceinline__ void gelu_erf_pair(float &x0, float &x1) {
    const uint64_t x = pk2(x0, x1);
    const uint64_t z = mul2(x, splat2(0.7071067811865476f));
    const uint64_t az = z & 0x7FFFFFFF7FFFFFFFull;
    float d0, d1;
    upk2(fma2(az, splat2(0.3275911f), splat2(1.0f)), d0, d1);
    const uint64_t t = pk2(rcp_approx(d0), rcp_approx(d1));
    // -(a1 t + a2 t^2 + a3 t^3 + a4 t^4 + a5 t^5)
    uint64_t poly = fma2(t, splat2(-1.061405429f), splat2(1.453152027f));
    poly = fma2(poly, t, splat2(-1.421413741f));
    poly = fma2(poly, t, splat2(0.284496736f));
    poly = fma2(poly, t, splat2(-0.254829592f));
    poly = mul2(poly, t);
    float e0, e1;
    upk2(mul2(mul2(az, az), splat2(-1.4426950408889634f)), e0, e1);
    const uint64_t e = pk2(ex2_approx(e0), ex2_approx(e1));
    uint64_t erf = fma2(poly, e, splat2(1.0f));                  // erf(|z|) >= 0
    erf |= z & 0x8000000080000000ull;                            // sign of z
    const uint64_t phi = fma2(erf, splat2(0.5f), splat2(0.5f));
    upk2(mul2(x, phi), x0, x1);
}

// 32-byte global accesses (sm_100): half as many memory instructions and L1 wavefronts per row as
// 16-byte ones.  The address must be 32-byte aligned.
__device__ __forceinline__ void st_global_32B(void *p, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t a4, uint32_t a5, uint32_t a6, uint32_t a7) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(a0), "r"(a1), "r"(a2),
                 "r"(a3), "r"(a4), "r"(a5), "r"(a6), "r"(a7)
                 : "memory");
}
__device__ __forceinline__ void ld_global_32B(const void *p, float (&r)[8]) {
    asm volatile("ld.global.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7])
                 : "l"(p)
                 : "memory");
}

__device__ __forceinline__ void store_bf16_chunk(uint16_t *dst, const float (&v)[32], int ncols) {
    if (ncols == 32 && (reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {
#pragma unroll
        for (int i = 0; i < 2; ++i)
            st_global_32B(dst + 16 * i, pack_h16x2(v[16 * i + 0], v[16 * i + 1]), pack_h16x2(v[16 * i + 2], v[16 * i + 3]),
                          pack_h16x2(v[16 * i + 4], v[16 * i + 5]), pack_h16x2(v[16 * i + 6], v[16 * i + 7]),
                          pack_h16x2(v[16 * i + 8], v[16 * i + 9]), pack_h16x2(v[16 * i + 10], v[16 * i + 11]),
                          pack_h16x2(v[16 * i + 12], v[16 * i + 13]), pack_h16x2(v[16 * i + 14], v[16 * i + 15]));
    } else if (ncols == 32 && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
        uint4 *d4 = reinterpret_cast<uint4 *>(dst);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint4 u;
            u.x = pack_h16x2(v[8 * i + 0], v[8 * i + 1]);
            u.y = pack_h16x2(v[8 * i + 2], v[8 * i + 3]);
            u.z = pack_h16x2(v[8 * i + 4], v[8 * i + 5]);
            u.w = pack_h16x2(v[8 * i + 6], v[8 * i + 7]);
            d4[i] = u;
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (i < ncols) dst[i] = to_h16((v[i]));
    }
}

__device__ __forceinline__ void store_f32_chunk(float *dst, const float (&v)[32], int ncols) {
    if (ncols == 32 && (reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            st_global_32B(dst + 8 * i, __float_as_uint(v[8 * i]), __float_as_uint(v[8 * i + 1]),
                          __float_as_uint(v[8 * i + 2]), __float_as_uint(v[8 * i + 3]), __float_as_uint(v[8 * i + 4]),
                          __float_as_uint(v[8 * i + 5]), __float_as_uint(v[8 * i + 6]), __float_as_uint(v[8 * i + 7]));
    } else if (ncols == 32 && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
        float4 *d4 = reinterpret_cast<float4 *>(dst);
#pragma unroll
        for (int i = 0; i < 8; ++i) d4[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (i < ncols) dst[i] = v[i];
    }
}

__device__ __forceinline__ void add_f32_chunk(const float *src, float (&v)[32], int ncols) {
    if (ncols == 32 && (reinterpret_cast<uintptr_t>(src) & 31u) == 0) {
        float t[4][8];
#pragma unroll
        for (int i = 0; i < 4; ++i) ld_global_32B(src + 8 * i, t[i]);
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) v[8 * i + j] += t[i][j];
    } else if (ncols == 32 && (reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
        const float4 *s4 = reinterpret_cast<const float4 *>(src);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float4 t = s4[i];
            v[4 * i] += t.x;
            v[4 * i + 1] += t.y;
            v[4 * i + 2] += t.z;
            v[4 * i + 3] += t.w;
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (i < ncols) v[i] += src[i];
    }
}

__device__ __forceinline__ void add_bias_chunk(const uint16_t *bias, float (&v)[32], int ncols) {
    if (ncols == 32 && (reinterpret_cast<uintptr_t>(bias) & 15u) == 0) {
        const uint4 *b4 = reinterpret_cast<const uint4 *>(bias);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint4 u = __ldg(b4 + i);
            v[8 * i + 0] += h16_lo(u.x);
            v[8 * i + 1] += h16_hi(u.x);
            v[8 * i + 2] += h16_lo(u.y);
            v[8 * i + 3] += h16_hi(u.y);
            v[8 * i + 4] += h16_lo(u.z);
            v[8 * i + 5] += h16_hi(u.z);
            v[8 * i + 6] += h16_lo(u.w);
            v[8 * i + 7] += h16_hi(u.w);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (i < ncols) v[i] += from_h16(bias[i]);
    }
}

// The same sums with the 32 bias values in shared memory (16-byte aligned; every lane reads the same words).
__device__ __forceinline__ void add_bias_chunk_parked(const uint16_t *bias, float (&v)[32]) {
    const uint4 *b4 = reinterpret_cast<const uint4 *>(bias);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint4 u = b4[i];
        v[8 * i + 0] += h16_lo(u.x);
        v[8 * i + 1] += h16_hi(u.x);
        v[8 * i + 2] += h16_lo(u.y);
        v[8 * i + 3] += h16_hi(u.y);
        v[8 * i + 4] += h16_lo(u.z);
        v[8 * i + 5] += h16_hi(u.z);
        v[8 * i + 6] += h16_lo(u.w);
        v[8 * i + 7] += h16_hi(u.w);
    }
}

// A warp parks 128 bias values (those past n_out as zeros) in its shared-memory strip while the MMAs of its tile
// run; lane l brings values 4 l .. 4 l + 3 of the strip, the bias of columns c .. c + 3.  A load from global memory
// per 32-column chunk, between the accumulator and the store, cost the chunk about 700 cycles (measured: 16-bit
// epilogue of a 128 x 256 tile 3.2 -> 2.6 us).
__device__ __forceinline__ void park_bias(const uint16_t *bias, int c, int n_out, uint16_t *strip, int lane) {
    uint2 b = make_uint2(0u, 0u);
    if (c + 4 <= n_out && (reinterpret_cast<uintptr_t>(bias + c) & 7u) == 0) {
        b = __ldg(reinterpret_cast<const uint2 *>(bias + c));
    } else {
        uint32_t e[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) e[i] = c + i < n_out ? bias[c + i] : 0u;
        b = make_uint2(e[0] | (e[1] << 16), e[2] | (e[3] << 16));
    }
    reinterpret_cast<uint2 *>(strip)[lane] = b;
    __syncwarp();
}

// One thread finishes 32 consecutive columns (col0 .. col0+31, the first ncols of them valid)
// of output row `row` of group g.  For KRAKEN_EPI_RESID_SUM the same thread must see the
// groups of one (row, column) in ascending order (the running sum is read back by its writer).
// with_bias = false: the caller has added the bias already.
__device__ __forceinline__ void epilogue_chunk(const EpiParams &p, int g, int row, int col0, int ncols,
                                               float (&v)[32], bool with_bias = true) {
    if (with_bias && p.bias) add_bias_chunk(p.bias + g * p.bias_gstride + col0, v, ncols);
    switch (p.kind) {
        case KRAKEN_EPI_F32:
            store_f32_chunk(p.out_f32 + g * p.out_f32_gstride + (long long)row * p.ld_out_f32 + col0, v, ncols);
            break;
        case KRAKEN_EPI_BF16:
            store_bf16_chunk(p.out_bf16 + g * p.out_bf16_gstride + (long long)row * p.ld_out_bf16 + col0, v, ncols);
            break;
        case KRAKEN_EPI_GELU_BF16:
            if (p.gelu_tanh) {
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = gelu_f(v[i], 1);
            } else {
#pragma unroll
                for (int i = 0; i < 32; i += 2) gelu_erf_pair(v[i], v[i + 1]);
            }
            store_bf16_chunk(p.out_bf16 + g * p.out_bf16_gstride + (long long)row * p.ld_out_bf16 + col0, v, ncols);
            break;
        case KRAKEN_EPI_RESID_F32:
            add_f32_chunk(p.resid + g * p.resid_gstride + (long long)row * p.ld_resid + col0, v, ncols);
            store_f32_chunk(p.out_f32 + g * p.out_f32_gstride + (long long)row * p.ld_out_f32 + col0, v, ncols);
            break;
        case KRAKEN_EPI_RESID_SUM: {
            add_f32_chunk(p.resid + g * p.resid_gstride + (long long)row * p.ld_resid + col0, v, ncols);
            store_f32_chunk(p.out_f32 + g * p.out_f32_gstride + (long long)row * p.ld_out_f32 + col0, v, ncols);
            float *s = p.sum + (long long)row * p.ld_sum + col0;
            if (g > 0) add_f32_chunk(s, v, ncols);
            store_f32_chunk(s, v, ncols);
            break;
        }
        case KRAKEN_EPI_QKV: {
            // columns [0, d) are q, the next n_kv_head * head_dim the key row, the last n_kv_head * head_dim the
            // value row of this token; keys and values go to their (sequence, head, position) row of the cache
            const int d = p.d_model;
            const int kvd = p.n_kv_head * p.head_dim;      // width of the k part and of the v part
            const int b = p.row_seq ? p.row_seq[row] : row / p.seqlen;
            const int pos = p.row_pos ? p.row_pos[row] : (p.pos0_dev ? p.pos0_dev[b] : p.pos0) + row % p.seqlen;
            if (((d | p.head_dim) & 31) == 0) {            // the 32 columns lie inside q or inside one head
                if (col0 < d) {
                    store_bf16_chunk(p.out_bf16 + g * p.out_bf16_gstride + (long long)row * p.ld_out_bf16 + col0, v,
                                     ncols);
                } else {
                    const int which = col0 >= d + kvd;
                    const int c = col0 - d - which * kvd;
                    const int head = c / p.head_dim, e0 = c % p.head_dim;
                    uint16_t *base = (which ? p.v_cache : p.k_cache) + g * p.cache_gstride;
                    store_bf16_chunk(base + (((long long)b * p.n_kv_head + head) * p.max_pos + pos) * p.head_dim + e0, v,
                                     ncols);
                }
            } else {
                // d_model and head_dim multiples of 8 only: 16-byte pieces, each inside q or one head
                // (ncols is a multiple of 8 because 3 d_model is)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (8 * i >= ncols) break;
                    const int col = col0 + 8 * i;
                    uint16_t *dst;
                    if (col < d) {
                        dst = p.out_bf16 + g * p.out_bf16_gstride + (long long)row * p.ld_out_bf16 + col;
                    } else {
                        const int which = col >= d + kvd;
                        const int c = col - d - which * kvd;
                        const int head = c / p.head_dim, e0 = c % p.head_dim;
                        dst = (which ? p.v_cache : p.k_cache) + g * p.cache_gstride +
                              (((long long)b * p.n_kv_head + head) * p.max_pos + pos) * p.head_dim + e0;
                    }
                    uint4 u;
                    u.x = pack_h16x2(v[8 * i + 0], v[8 * i + 1]);
                    u.y = pack_h16x2(v[8 * i + 2], v[8 * i + 3]);
                    u.z = pack_h16x2(v[8 * i + 4], v[8 * i + 5]);
                    u.w = pack_h16x2(v[8 * i + 6], v[8 * i + 7]);
                    *reinterpret_cast<uint4 *>(dst) = u;
                }
            }
            break;
        }
        default:
            break;
    }
}

// fp32 epilogues (plain, + residual, + residual and cross-branch sum) of one warp's 32 rows x 32
// columns with fully coalesced global accesses.  Thread = row cannot coalesce (32 rows per instruction,
// one L1 wavefront per row piece, and the epilogue warps of an SM share one load/store pipe), so each
// thread parks its row in a per-warp shared-memory tile (pitch 36 floats: conflict-free 16-byte
// accesses both ways) and the warp then walks the tile 4 rows x 128 bytes per instruction.
// The bias has already been added.  Rows must be 16-byte aligned.  The (warp, lane) -> (row, column)
// mapping is fixed, which keeps the running sum of KRAKEN_EPI_RESID_SUM on the thread that wrote it.
constexpr int EPI_STAGE_PITCH = 36;
constexpr int EPI_STAGE_FLOATS = 32 * EPI_STAGE_PITCH;

// With `ln` set (LayerNorm fused behind the epilogue) the finished row, plus ln_y, comes back in v in the
// thread = row mapping, for the row statistics and for the copy kept in tensor memory.
__device__ __forceinline__ void epilogue_f32_staged(const EpiParams &p, int g, int row_base, int m, int col0,
                                                    float (&v)[32], float *stage, int lane, bool ln = false) {
    float4 *mine = reinterpret_cast<float4 *>(stage + lane * EPI_STAGE_PITCH);
#pragma unroll
    for (int j = 0; j < 8; ++j) mine[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
    __syncwarp();
    const int r_in = lane >> 3, c4 = (lane & 7) << 2;
    const long long col = col0 + c4;
    // all loads of a phase are issued before any store: the pointers may alias as far as the compiler
    // knows, so a store in between would serialise the loads behind it
    float4 x[8];
#pragma unroll
    for (int it = 0; it < 8; ++it)
        x[it] = *reinterpret_cast<const float4 *>(stage + (it * 4 + r_in) * EPI_STAGE_PITCH + c4);
    if (p.kind != KRAKEN_EPI_F32) {
        float4 t[8];
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int row = row_base + it * 4 + r_in;
            t[it] = row < m ? *reinterpret_cast<const float4 *>(p.resid + g * p.resid_gstride +
                                                                (long long)row * p.ld_resid + col)
                            : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            x[it].x += t[it].x; x[it].y += t[it].y; x[it].z += t[it].z; x[it].w += t[it].w;
        }
    }
    if (p.kind == KRAKEN_EPI_RESID_SUM && g > 0) {
        float4 t[8];
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int row = row_base + it * 4 + r_in;
            t[it] = row < m ? *reinterpret_cast<const float4 *>(p.sum + (long long)row * p.ld_sum + col)
                            : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int row = row_base + it * 4 + r_in;
            if (row < m) {
                *reinterpret_cast<float4 *>(p.out_f32 + g * p.out_f32_gstride + (long long)row * p.ld_out_f32 + col) = x[it];
                t[it].x += x[it].x; t[it].y += x[it].y; t[it].z += x[it].z; t[it].w += x[it].w;
                *reinterpret_cast<float4 *>(p.sum + (long long)row * p.ld_sum + col) = t[it];
            }
        }
    } else {
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int row = row_base + it * 4 + r_in;
            if (row < m) {
                *reinterpret_cast<float4 *>(p.out_f32 + g * p.out_f32_gstride + (long long)row * p.ld_out_f32 + col) = x[it];
                if (p.kind == KRAKEN_EPI_RESID_SUM)
                    *reinterpret_cast<float4 *>(p.sum + (long long)row * p.ld_sum + col) = x[it];
            }
        }
    }
    __syncwarp();
    if (ln) {
        if (p.ln_y) {
#pragma unroll
            for (int it = 0; it < 8; ++it) {
                const int row = row_base + it * 4 + r_in;
                if (row < m) {
                    const float4 y = *reinterpret_cast<const float4 *>(p.ln_y + (long long)row * p.ln_ld_y + col);
                    x[it].x += y.x; x[it].y += y.y; x[it].z += y.z; x[it].w += y.w;
                }
            }
        }
#pragma unroll
        for (int it = 0; it < 8; ++it)
            *reinterpret_cast<float4 *>(stage + (it * 4 + r_in) * EPI_STAGE_PITCH + c4) = x[it];
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float4 r = mine[j];
            v[4 * j] = r.x; v[4 * j + 1] = r.y; v[4 * j + 2] = r.z; v[4 * j + 3] = r.w;
        }
        __syncwarp();
    }
}

// ---------------------------------------------------------------- LayerNorm fused behind the fp32 epilogues
// (Algorithm 1: x = LN(x) after `out = res + FFN(x)`, x = LN(x + y) after `x = res + MHA(x)`.)

// Running (mean, M2, count) of one row, updated with up to 32 new values: the values are centred on
// their own mean first and the two sets are joined with the pairwise update, so nothing cancels.
struct RowStats {
    float mean, m2, cnt;
};

__device__ __forceinline__ void stats_join(RowStats &s, float mean_b, float m2_b, float n_b) {
    if (n_b == 0.f) return;
    const float tot = s.cnt + n_b;
    const float delta = mean_b - s.mean;
    const float w = n_b / tot;
    s.mean = fmaf(delta, w, s.mean);
    s.m2 += m2_b + delta * delta * s.cnt * w;
    s.cnt = tot;
}

__device__ __forceinline__ void stats_add_chunk(RowStats &s, const float (&z)[32], int ncols) {
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
        a0 += i < ncols ? z[i] : 0.f;
        a1 += i + 1 < ncols ? z[i + 1] : 0.f;
        a2 += i + 2 < ncols ? z[i + 2] : 0.f;
        a3 += i + 3 < ncols ? z[i + 3] : 0.f;
    }
    const float cm = ((a0 + a1) + (a2 + a3)) / static_cast<float>(ncols);
    float q0 = 0.f, q1 = 0.f, q2 = 0.f, q3 = 0.f;
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
        const float d0 = z[i] - cm, d1 = z[i + 1] - cm, d2 = z[i + 2] - cm, d3 = z[i + 3] - cm;
        q0 = i < ncols ? fmaf(d0, d0, q0) : q0;
        q1 = i + 1 < ncols ? fmaf(d1, d1, q1) : q1;
        q2 = i + 2 < ncols ? fmaf(d2, d2, q2) : q2;
        q3 = i + 3 < ncols ? fmaf(d3, d3, q3) : q3;
    }
    stats_join(s, cm, (q0 + q1) + (q2 + q3), static_cast<float>(ncols));
}

__device__ __forceinline__ void load_h16_chunk(const uint16_t *src, float (&o)[32], int ncols, float fill) {
    if (ncols == 32 && (reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
        const uint4 *b4 = reinterpret_cast<const uint4 *>(src);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint4 u = __ldg(b4 + i);
            o[8 * i + 0] = h16_lo(u.x); o[8 * i + 1] = h16_hi(u.x);
            o[8 * i + 2] = h16_lo(u.y); o[8 * i + 3] = h16_hi(u.y);
            o[8 * i + 4] = h16_lo(u.z); o[8 * i + 5] = h16_hi(u.z);
            o[8 * i + 6] = h16_lo(u.w); o[8 * i + 7] = h16_hi(u.w);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = i < ncols ? from_h16(src[i]) : fill;
    }
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// The warp has left its part of 32 rows in ln_parts: count it in, then wait until all `need` parts of those
// rows are there.  Bounded like every other wait; false = gave up (abort flag raised).
__device__ __forceinline__ bool ln_arrive_and_wait(uint32_t *cnt, uint32_t need, int lane, volatile uint32_t *abort_flag) {
    __threadfence();
    __syncwarp();
    bool ok = true;
    if (lane == 0) {
        atomicAdd(cnt, 1u);
        unsigned long long t0 = 0;
        uint32_t polls = 0;
        while (ld_acquire_u32(cnt) < need) {
            __nanosleep(40);
            if ((++polls & 63u) == 0u) {
                if (*abort_flag) { ok = false; break; }
                const unsigned long long now = global_timer_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > WAIT_LIMIT_NS) { *abort_flag = 1u; ok = false; break; }
            }
        }
    }
    // lane 0's acquire and the warp barrier order the other lanes' reads of the parts (which bypass L1) behind it
    ok = __all_sync(0xFFFFFFFFu, ok);
    return ok;
}

// The last of the `need` warps to leave a slab of rows puts its two counters back to zero for the next launch.
__device__ __forceinline__ void ln_depart(uint32_t *cnt, uint32_t need, int lane) {
    __syncwarp();
    if (lane == 0) {
        if (atomicAdd(cnt + 1, 1u) == need - 1u) {
            cnt[0] = 0u;
            cnt[1] = 0u;
        }
    }
}

// Joins the parts of one row in their fixed order: mean and 1 / sqrt(var + eps) of the whole row.
__device__ __forceinline__ void ln_row_stats(const float4 *parts, int n_parts, float eps, float &mean, float &rstd) {
    RowStats s{0.f, 0.f, 0.f};
    for (int p0 = 0; p0 < n_parts; p0 += 8) {      // eight loads in flight, then joined in order
        float4 v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = p0 + i < n_parts ? __ldcg(parts + p0 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 8; ++i) stats_join(s, v[i].x, v[i].y, v[i].z);
    }
    mean = s.mean;
    rstd = rsqrtf(s.m2 / s.cnt + eps);
}

// Second pass over one 32-column chunk of one row (the thread's own TMEM lane): normalise and store 16-bit.
__device__ __forceinline__ void ln_store_chunk(const EpiParams &p, int g, int row, int col0, int ncols, float (&z)[32],
                                               float mean, float rstd) {
    float gam[32], bet[32];
    load_h16_chunk(p.ln_gamma + g * p.ln_gb_gstride + col0, gam, ncols, 0.f);
    if (p.ln_beta) load_h16_chunk(p.ln_beta + g * p.ln_gb_gstride + col0, bet, ncols, 0.f);
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        const float n = (z[i] - mean) * rstd;
        z[i] = p.ln_beta ? fmaf(n, gam[i], bet[i]) : n * gam[i];
    }
    store_bf16_chunk(p.ln_out + g * p.ln_out_gstride + (long long)row * p.ln_ld_out + col0, z, ncols);
}

// The thread = row form of the fp32 epilogues with a LayerNorm behind them (one thread finishes 32 columns of
// its row): bias, residual, the fp32 output, the running cross-branch sum; v comes back as the row the
// LayerNorm sees (out + ln_y).
__device__ __forceinline__ void epilogue_chunk_ln(const EpiParams &p, int g, int row, int col0, int ncols,
                                                  float (&v)[32]) {
    if (p.bias) add_bias_chunk(p.bias + g * p.bias_gstride + col0, v, ncols);
    add_f32_chunk(p.resid + g * p.resid_gstride + (long long)row * p.ld_resid + col0, v, ncols);
    store_f32_chunk(p.out_f32 + g * p.out_f32_gstride + (long long)row * p.ld_out_f32 + col0, v, ncols);
    if (p.kind == KRAKEN_EPI_RESID_SUM) {
        float t[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) t[i] = v[i];
        float *sp = p.sum + (long long)row * p.ld_sum + col0;
        if (g > 0) add_f32_chunk(sp, t, ncols);
        store_f32_chunk(sp, t, ncols);
    }
    if (p.ln_y) add_f32_chunk(p.ln_y + (long long)row * p.ln_ld_y + col0, v, ncols);
}

__device__ __forceinline__ bool epilogue_f32_stageable(const EpiParams &p) {
    if (p.kind != KRAKEN_EPI_F32 && p.kind != KRAKEN_EPI_RESID_F32 && p.kind != KRAKEN_EPI_RESID_SUM) return false;
    bool ok = (p.ld_out_f32 & 3) == 0 && (reinterpret_cast<uintptr_t>(p.out_f32) & 15) == 0 &&
              (p.out_f32_gstride & 3) == 0;
    if (p.kind != KRAKEN_EPI_F32)
        ok = ok && (p.ld_resid & 3) == 0 && (reinterpret_cast<uintptr_t>(p.resid) & 15) == 0 &&
             (p.resid_gstride & 3) == 0;
    if (p.kind == KRAKEN_EPI_RESID_SUM) ok = ok && (p.ld_sum & 3) == 0 && (reinterpret_cast<uintptr_t>(p.sum) & 15) == 0;
    if (p.ln_out && p.ln_y) ok = ok && (p.ln_ld_y & 3) == 0 && (reinterpret_cast<uintptr_t>(p.ln_y) & 15) == 0;
    return ok;
}

}  // namespace kr
