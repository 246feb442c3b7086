// HBM-bound steps of the path: shared embedding, the two LayerNorms of Algorithm 1 (the second
// one fused with the addition of the cross-branch sum y), and the W_concat input gather.
// One warp per row, 16-byte loads and stores, statistics in fp32.
#include "internal.h"
#include "ptx.cuh"

namespace kr {

namespace {

constexpr int ROW_WARPS = 8;  // warps (rows) per CTA

__global__ void __launch_bounds__(ROW_WARPS * 32)
embed_kernel(const int32_t *__restrict__ ids, int n_tokens, int seqlen, int pos0, const uint16_t *__restrict__ wte,
             const uint16_t *__restrict__ wpe, int d, int vocab, float *__restrict__ out, uint32_t *status,
             const int *__restrict__ pos0_dev, const int *__restrict__ row_pos) {
    pdl_wait();
    pdl_trigger();
    const int t = blockIdx.x * ROW_WARPS + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (t >= n_tokens) return;
    int id = ids[t];
    if (id < 0 || id >= vocab) {
        if (lane == 0 && status) atomicOr(status, STATUS_BAD_TOKEN);
        id = 0;
    }
    // position: from the packed-batch table, else the sequence's first position (device array or host value)
    // plus the offset inside the sequence
    const int pos = row_pos ? row_pos[t] : (pos0_dev ? pos0_dev[t / seqlen] : pos0) + t % seqlen;
    const uint4 *te = reinterpret_cast<const uint4 *>(wte + (size_t)id * d);
    const uint4 *pe = reinterpret_cast<const uint4 *>(wpe + (size_t)pos * d);
    float4 *o = reinterpret_cast<float4 *>(out + (size_t)t * d);
    for (int v = lane; v < d / 8; v += 32) {
        const uint4 a = __ldg(te + v), b = __ldg(pe + v);
        o[2 * v] = make_float4(h16_lo(a.x) + h16_lo(b.x), h16_hi(a.x) + h16_hi(b.x),
                               h16_lo(a.y) + h16_lo(b.y), h16_hi(a.y) + h16_hi(b.y));
        o[2 * v + 1] = make_float4(h16_lo(a.z) + h16_lo(b.z), h16_hi(a.z) + h16_hi(b.z),
                                   h16_lo(a.w) + h16_lo(b.w), h16_hi(a.w) + h16_hi(b.w));
    }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}


// out[g][r, :] = bf16( gamma_g * (v - mean) * rstd + beta_g ),  v = a[g][r, :] + y[r, :]
// where y is absent, a given [rows, d] tensor, or the sum over `ysum_groups` tensors taken in
// ascending order (the cross-branch sum computed on the fly when the row count is small).
// LN_CACHE: float4 per lane kept in registers (16: rows up to 2048 wide in one pass; 8: up to 1024,
// with half the registers and twice the resident warps)
// DENSE: without the code for summing the branch inputs and capped at 64 registers, so that four CTAs fit an SM, for
// launches of more CTAs than three per SM (4096 rows of 1024: 8.8 -> 5.7 us).  Launches of few rows keep the full
// build: a decode step measured 4 % slower with the trimmed one.
template <int LN_CACHE, bool YSUM, bool DENSE = false>
__global__ void __launch_bounds__(ROW_WARPS * 32, LN_CACHE == 8 ? (DENSE ? 4 : 2) : 0)
layernorm_kernel(const float *__restrict__ a, long long a_gstride, const float *__restrict__ y,
                 const float *__restrict__ ysum, long long ysum_gstride, int ysum_groups,
                 const uint16_t *__restrict__ gamma, const uint16_t *__restrict__ beta, int groups, int rows, int d,
                 float eps, uint16_t *__restrict__ out) {
    pdl_wait();
    const long long wr = (long long)blockIdx.x * ROW_WARPS + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (wr >= (long long)groups * rows) return;
    // neighbouring warps take the groups of one row, so the shared y row is fetched from DRAM once
    const int r = static_cast<int>(wr / groups), g = static_cast<int>(wr % groups);
    const float4 *pa = reinterpret_cast<const float4 *>(a + g * a_gstride + (size_t)r * d);
    const float4 *py = y ? reinterpret_cast<const float4 *>(y + (size_t)r * d) : nullptr;
    const float4 *ps = (YSUM && ysum) ? reinterpret_cast<const float4 *>(ysum + (size_t)r * d) : nullptr;
    const int nvec = d / 4;

    auto load = [&](int v) {
        float4 t = pa[v];
        if (py) {
            const float4 u = py[v];
            t.x += u.x; t.y += u.y; t.z += u.z; t.w += u.w;
        } else if (YSUM && ps) {
            float4 acc = ps[v];
            for (int m = 1; m < ysum_groups; ++m) {
                const float4 u = ps[(size_t)m * (ysum_gstride / 4) + v];
                acc.x += u.x; acc.y += u.y; acc.z += u.z; acc.w += u.w;
            }
            t.x += acc.x; t.y += acc.y; t.z += acc.z; t.w += acc.w;
        }
        return t;
    };

    // Launches of few rows (a decode step) are a chain of dependent round trips to L2; there gamma and beta are
    // requested together with the row instead of after the statistics.
    constexpr bool EARLY_GB = LN_CACHE == 8 && !DENSE;
    const uint2 *pg = nullptr, *pb = nullptr;
    uint2 gmc[EARLY_GB ? LN_CACHE : 1], btc[EARLY_GB ? LN_CACHE : 1];
    if (EARLY_GB) {
        pg = reinterpret_cast<const uint2 *>(gamma + (size_t)g * d);
        pb = beta ? reinterpret_cast<const uint2 *>(beta + (size_t)g * d) : nullptr;
#pragma unroll
        for (int i = 0; i < LN_CACHE; ++i) {
            const int v = lane + 32 * i;
            gmc[EARLY_GB ? i : 0] = v < nvec ? __ldg(pg + v) : make_uint2(0u, 0u);
            btc[EARLY_GB ? i : 0] = (pb && v < nvec) ? __ldg(pb + v) : make_uint2(0u, 0u);
        }
    }
    float4 cache[LN_CACHE];
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < LN_CACHE; ++i) {
        const int v = lane + 32 * i;
        if (v < nvec) {
            const float4 t = load(v);
            cache[i] = t;
            sum += (t.x + t.y) + (t.z + t.w);
        }
    }
    for (int v = lane + 32 * LN_CACHE; v < nvec; v += 32) {
        const float4 t = load(v);
        sum += (t.x + t.y) + (t.z + t.w);
    }
    const float mean = warp_sum(sum) / d;
    float sq = 0.f;
#pragma unroll
    for (int i = 0; i < LN_CACHE; ++i) {
        const int v = lane + 32 * i;
        if (v < nvec) {
            const float4 t = cache[i];
            const float dx = t.x - mean, dy = t.y - mean, dz = t.z - mean, dw = t.w - mean;
            sq += (dx * dx + dy * dy) + (dz * dz + dw * dw);
        }
    }
    for (int v = lane + 32 * LN_CACHE; v < nvec; v += 32) {
        const float4 t = load(v);
        const float dx = t.x - mean, dy = t.y - mean, dz = t.z - mean, dw = t.w - mean;
        sq += (dx * dx + dy * dy) + (dz * dz + dw * dw);
    }
    const float rstd = rsqrtf(warp_sum(sq) / d + eps);
    pdl_trigger();

    if (!EARLY_GB) {
        pg = reinterpret_cast<const uint2 *>(gamma + (size_t)g * d);
        pb = beta ? reinterpret_cast<const uint2 *>(beta + (size_t)g * d) : nullptr;
    }
    uint2 *po = reinterpret_cast<uint2 *>(out + ((size_t)g * rows + r) * d);
    auto emit_gb = [&](int v, const float4 &t, const uint2 gm, const uint2 bt) {
        const float o0 = (t.x - mean) * rstd * h16_lo(gm.x) + h16_lo(bt.x);
        const float o1 = (t.y - mean) * rstd * h16_hi(gm.x) + h16_hi(bt.x);
        const float o2 = (t.z - mean) * rstd * h16_lo(gm.y) + h16_lo(bt.y);
        const float o3 = (t.w - mean) * rstd * h16_hi(gm.y) + h16_hi(bt.y);
        po[v] = make_uint2(pack_h16x2(o0, o1), pack_h16x2(o2, o3));
    };
    auto emit = [&](int v, const float4 &t) {
        emit_gb(v, t, __ldg(pg + v), pb ? __ldg(pb + v) : make_uint2(0u, 0u));
    };
#pragma unroll
    for (int i = 0; i < LN_CACHE; ++i) {
        const int v = lane + 32 * i;
        if (v < nvec) {
            if (EARLY_GB) emit_gb(v, cache[i], gmc[EARLY_GB ? i : 0], btc[EARLY_GB ? i : 0]);
            else emit(v, cache[i]);
        }
    }
    for (int v = lane + 32 * LN_CACHE; v < nvec; v += 32) emit(v, load(v));
}

// The same LayerNorm with one CTA per row: for rows wider than a warp can keep in registers (d > 2048, where the
// kernel above goes over the tail of the row three times) and for few, wide rows, where eight warps on one row
// shorten the chain of dependent memory round trips that a single warp would walk alone.  Thread t holds elements
// 4 (t + 256 i) .. + 3; partial sums go through a warp shuffle tree and then through shared memory, added in warp
// order by every thread, so the result does not depend on timing.
constexpr int LNB_THREADS = 256;
constexpr int LNB_CACHE = 8;   // float4 per thread: rows up to 8192 wide

__global__ void __launch_bounds__(LNB_THREADS, 4)
layernorm_block_kernel(const float *__restrict__ a, long long a_gstride, const float *__restrict__ y,
                       const uint16_t *__restrict__ gamma, const uint16_t *__restrict__ beta, int groups, int rows,
                       int d, float eps, uint16_t *__restrict__ out) {
    __shared__ float red[2][LNB_THREADS / 32];
    pdl_wait();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nvec = d / 4;
    bool triggered = false;
    for (long long wr = blockIdx.x; wr < (long long)groups * rows; wr += gridDim.x) {
        // neighbouring CTAs take the groups of one row, so the shared y row is fetched from DRAM once
        const int r = static_cast<int>(wr / groups), g = static_cast<int>(wr % groups);
        const float4 *pa = reinterpret_cast<const float4 *>(a + g * a_gstride + (size_t)r * d);
        const float4 *py = y ? reinterpret_cast<const float4 *>(y + (size_t)r * d) : nullptr;
        float4 cache[LNB_CACHE];
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < LNB_CACHE; ++i) {
            const int v = tid + LNB_THREADS * i;
            if (v < nvec) {
                float4 t = pa[v];
                if (py) {
                    const float4 u = py[v];
                    t.x += u.x; t.y += u.y; t.z += u.z; t.w += u.w;
                }
                cache[i] = t;
                sum += (t.x + t.y) + (t.z + t.w);
            }
        }
        sum = warp_sum(sum);
        if (lane == 0) red[0][warp] = sum;
        __syncthreads();
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < LNB_THREADS / 32; ++w) tot += red[0][w];
        const float mean = tot / d;
        float sq = 0.f;
#pragma unroll
        for (int i = 0; i < LNB_CACHE; ++i) {
            const int v = tid + LNB_THREADS * i;
            if (v < nvec) {
                const float4 t = cache[i];
                const float dx = t.x - mean, dy = t.y - mean, dz = t.z - mean, dw = t.w - mean;
                sq += (dx * dx + dy * dy) + (dz * dz + dw * dw);
            }
        }
        sq = warp_sum(sq);
        if (lane == 0) red[1][warp] = sq;
        __syncthreads();
        float tot2 = 0.f;
#pragma unroll
        for (int w = 0; w < LNB_THREADS / 32; ++w) tot2 += red[1][w];
        const float rstd = rsqrtf(tot2 / d + eps);
        if (!triggered) {
            pdl_trigger();
            triggered = true;
        }
        const uint2 *pg = reinterpret_cast<const uint2 *>(gamma + (size_t)g * d);
        const uint2 *pb = beta ? reinterpret_cast<const uint2 *>(beta + (size_t)g * d) : nullptr;
        uint2 *po = reinterpret_cast<uint2 *>(out + ((size_t)g * rows + r) * d);
#pragma unroll
        for (int i = 0; i < LNB_CACHE; ++i) {
            const int v = tid + LNB_THREADS * i;
            if (v < nvec) {
                const float4 t = cache[i];
                const uint2 gm = __ldg(pg + v);
                uint2 bt = make_uint2(0u, 0u);
                if (pb) bt = __ldg(pb + v);
                const float o0 = (t.x - mean) * rstd * h16_lo(gm.x) + h16_lo(bt.x);
                const float o1 = (t.y - mean) * rstd * h16_hi(gm.x) + h16_hi(bt.x);
                const float o2 = (t.z - mean) * rstd * h16_lo(gm.y) + h16_lo(bt.y);
                const float o3 = (t.w - mean) * rstd * h16_hi(gm.y) + h16_hi(bt.y);
                po[v] = make_uint2(pack_h16x2(o0, o1), pack_h16x2(o2, o3));
            }
        }
        // red[] is written again by the next row only after every thread has passed the second barrier of
        // this one; its first barrier then keeps the two rows' partial sums apart
    }
    if (!triggered) pdl_trigger();
}

// The same LayerNorm for many rows, as a persistent producer / consumer kernel: what limits the
// warp-per-row kernel above is that a warp has nothing in flight while it reduces and writes, so here
// one thread keeps a ring of whole rows in flight with bulk copies (a stage = the N group rows of one
// row index plus the shared y row, each fetched from DRAM once) and twelve (or up to sixteen) consumer warps take the rows
// out of shared memory into registers, release the stage at once and then reduce, normalise and store.
// Consumer warp c works on group c % groups of every (c / groups)-th stage; the number of stages is a
// multiple of the number of such warp sets, so a ring slot is always consumed by the same set and every
// waiter sees every phase of the barriers it waits on.
constexpr int LNS_CONSUMERS = 12;       // group counts that divide 12 (1, 2, 3, 4, 6, 12)
constexpr int LNS_CONSUMERS_WIDE = 16;  // other group counts up to 16: the largest multiple of the count <= 16
constexpr int LNS_MAX_STAGES = 12;
constexpr int LNS_SMEM_BUDGET = 226 * 1024;

template <int LN_CACHE, int MAX_CONSUMERS>
__global__ void __launch_bounds__((MAX_CONSUMERS + 1) * 32, 1)
layernorm_stream_kernel(const float *__restrict__ a, long long a_gstride, const float *__restrict__ y,
                        const uint16_t *__restrict__ gamma, const uint16_t *__restrict__ beta, int groups, int rows,
                        int d, float eps, uint16_t *__restrict__ out, int stages, int n_consumers, uint32_t *status) {
    extern __shared__ __align__(128) uint8_t lns_smem[];
    __shared__ uint64_t full[LNS_MAX_STAGES], empty[LNS_MAX_STAGES];
    __shared__ uint32_t abort_word;
    volatile uint32_t *abort_flag = &abort_word;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t row_bytes = static_cast<uint32_t>(d) * 4u;
    const uint32_t stage_bytes = row_bytes * (groups + (y ? 1 : 0));
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(full + s, 1);
            mbar_init(empty + s, groups);
        }
        abort_word = 0;
        fence_barrier_init();
    }
    // gamma and beta of every group sit behind the ring: with most of the SM's memory carved out as
    // shared memory the L1 left over does not hold them, and their latency would sit on every row
    uint16_t *s_gamma = reinterpret_cast<uint16_t *>(lns_smem + (size_t)stages * stage_bytes);
    uint16_t *s_beta = s_gamma + (size_t)groups * d;
    for (int i = threadIdx.x; i < groups * d / 4; i += blockDim.x) {
        reinterpret_cast<uint2 *>(s_gamma)[i] = __ldg(reinterpret_cast<const uint2 *>(gamma) + i);
        reinterpret_cast<uint2 *>(s_beta)[i] = beta ? __ldg(reinterpret_cast<const uint2 *>(beta) + i) : make_uint2(0u, 0u);
    }
    __syncthreads();
    pdl_wait();   // gamma and beta are weights; everything below touches what the predecessor wrote
    const int n_units = (rows - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);

    if (warp == n_consumers) {
        if (lane == 0) {
            for (int k = 0; k < n_units; ++k) {
                const int slot = k % stages;
                const size_t r = blockIdx.x + (size_t)k * gridDim.x;
                if (!mbar_wait(empty + slot, ((k / stages) & 1) ^ 1, abort_flag)) break;
                uint8_t *dst = lns_smem + (size_t)slot * stage_bytes;
                mbar_expect_tx(full + slot, stage_bytes);
                for (int g = 0; g < groups; ++g)
                    bulk_load(dst + g * row_bytes, a + g * a_gstride + r * d, row_bytes, full + slot);
                if (y) bulk_load(dst + groups * row_bytes, y + r * d, row_bytes, full + slot);
            }
        }
        __syncwarp();
    } else {
        const int n_sets = n_consumers / groups;
        const int set = warp / groups, g = warp % groups;
        const int nvec = d / 4;
        const uint2 *pg = reinterpret_cast<const uint2 *>(s_gamma + (size_t)g * d);
        const uint2 *pb = reinterpret_cast<const uint2 *>(s_beta + (size_t)g * d);
        for (int k = set; k < n_units; k += n_sets) {
            const int slot = k % stages;
            const size_t r = blockIdx.x + (size_t)k * gridDim.x;
            bool ok = mbar_wait(full + slot, (k / stages) & 1, abort_flag);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            const float4 *sa = reinterpret_cast<const float4 *>(lns_smem + (size_t)slot * stage_bytes + g * row_bytes);
            const float4 *sy = reinterpret_cast<const float4 *>(lns_smem + (size_t)slot * stage_bytes + groups * row_bytes);
            float4 cache[LN_CACHE];
            float sum = 0.f;
#pragma unroll
            for (int i = 0; i < LN_CACHE; ++i) {
                const int v = lane + 32 * i;
                if (v < nvec) {
                    float4 t = sa[v];
                    if (y) {
                        const float4 u = sy[v];
                        t.x += u.x; t.y += u.y; t.z += u.z; t.w += u.w;
                    }
                    cache[i] = t;
                    sum += (t.x + t.y) + (t.z + t.w);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty + slot);          // the row is in registers: the stage may be refilled
            const float mean = warp_sum(sum) / d;
            float sq = 0.f;
#pragma unroll
            for (int i = 0; i < LN_CACHE; ++i) {
                const int v = lane + 32 * i;
                if (v < nvec) {
                    const float4 t = cache[i];
                    const float dx = t.x - mean, dy = t.y - mean, dz = t.z - mean, dw = t.w - mean;
                    sq += (dx * dx + dy * dy) + (dz * dz + dw * dw);
                }
            }
            const float rstd = rsqrtf(warp_sum(sq) / d + eps);
            uint2 *po = reinterpret_cast<uint2 *>(out + ((size_t)g * rows + r) * d);
#pragma unroll
            for (int i = 0; i < LN_CACHE; ++i) {
                const int v = lane + 32 * i;
                if (v < nvec) {
                    const float4 t = cache[i];
                    const uint2 gm = pg[v];
                    const uint2 bt = pb[v];
                    const float o0 = (t.x - mean) * rstd * h16_lo(gm.x) + h16_lo(bt.x);
                    const float o1 = (t.y - mean) * rstd * h16_hi(gm.x) + h16_hi(bt.x);
                    const float o2 = (t.z - mean) * rstd * h16_lo(gm.y) + h16_lo(bt.y);
                    const float o3 = (t.w - mean) * rstd * h16_hi(gm.y) + h16_hi(bt.y);
                    po[v] = make_uint2(pack_h16x2(o0, o1), pack_h16x2(o2, o3));
                }
            }
        }
    }
    __syncthreads();
    if (*abort_flag) {
        // a wait ran out: give copies still in flight time to land before the shared memory is released
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
        if (threadIdx.x == 0 && status) atomicOr(status, STATUS_WAIT_LIMIT);
    }
}

__global__ void __launch_bounds__(ROW_WARPS * 32)
gather_concat_kernel(const float *__restrict__ x, long long x_gstride, int groups, int d,
                     const int32_t *__restrict__ rows, int n_rows, uint16_t *__restrict__ out) {
    pdl_wait();
    pdl_trigger();
    const long long w = (long long)blockIdx.x * ROW_WARPS + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (w >= (long long)n_rows * groups) return;
    const int r = static_cast<int>(w / groups), g = static_cast<int>(w % groups);
    const int src_row = rows ? rows[r] : r;
    const float4 *src = reinterpret_cast<const float4 *>(x + g * x_gstride + (size_t)src_row * d);
    uint2 *dst = reinterpret_cast<uint2 *>(out + ((size_t)r * groups + g) * d);
    for (int v = lane; v < d / 4; v += 32) {
        const float4 t = src[v];
        dst[v] = make_uint2(pack_h16x2(t.x, t.y), pack_h16x2(t.z, t.w));
    }
}

// dst[g][i][:] = src[g][rows[i]][:] for rows of row_bytes bytes (a multiple of 16), one warp per (group, row)
__global__ void __launch_bounds__(ROW_WARPS * 32)
gather_rows_kernel(const uint8_t *__restrict__ src, long long src_gstride, int groups, int row_bytes,
                   const int32_t *__restrict__ rows, int n_rows, uint8_t *__restrict__ dst) {
    pdl_wait();
    pdl_trigger();
    const long long w = (long long)blockIdx.x * ROW_WARPS + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (w >= (long long)n_rows * groups) return;
    const int r = static_cast<int>(w % n_rows), g = static_cast<int>(w / n_rows);
    const uint4 *s = reinterpret_cast<const uint4 *>(src + g * src_gstride + (size_t)rows[r] * row_bytes);
    uint4 *d = reinterpret_cast<uint4 *>(dst + ((size_t)g * n_rows + r) * row_bytes);
    for (int v = lane; v < row_bytes / 16; v += 32) d[v] = s[v];
}

// out = x_0 + x_1 + ... + x_{G-1} element by element, added in ascending group order (the order the
// down-projection epilogue and LayerNorm-2 use when they form the same cross-branch sum themselves)
__global__ void __launch_bounds__(256)
sum_groups_kernel(const float *__restrict__ x, long long gstride, int groups, long long n4, float *__restrict__ out) {
    pdl_wait();
    pdl_trigger();
    const float4 *px = reinterpret_cast<const float4 *>(x);
    float4 *po = reinterpret_cast<float4 *>(out);
    const long long stride = (long long)gridDim.x * blockDim.x, gs4 = gstride / 4;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
        float4 acc = px[i];
        for (int g = 1; g < groups; ++g) {
            const float4 t = px[g * gs4 + i];
            acc.x += t.x; acc.y += t.y; acc.z += t.z; acc.w += t.w;
        }
        po[i] = acc;
    }
}

__global__ void f32_to_bf16_kernel(const float *__restrict__ in, uint16_t *__restrict__ out, long long n) {
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (; i < n; i += stride) out[i] = to_h16((in[i]));
}

int done() { return cudaGetLastError() == cudaSuccess ? KRAKEN_OK : KRAKEN_ECUDA; }

}  // namespace

int launch_embed(const int32_t *ids, int n_tokens, int seqlen, int pos0, const uint16_t *wte, const uint16_t *wpe,
                 int d, int vocab, float *out, uint32_t *status, cudaStream_t stream, const int *pos0_dev,
                 const int *row_pos) {
    if (!ids || !wte || !wpe || !out || n_tokens < 1 || seqlen < 1 || pos0 < 0 || d < 8 || (d & 7) || vocab < 1)
        return KRAKEN_EINVAL;
    return cuda_check(launch_pdl(embed_kernel, dim3((n_tokens + ROW_WARPS - 1) / ROW_WARPS), dim3(ROW_WARPS * 32), 0,
                                 stream, ids, n_tokens, seqlen, pos0, wte, wpe, d, vocab, out, status, pos0_dev, row_pos),
                      "embed: launch");
}

// whether the persistent kernel takes the call: enough rows to fill its ring on every SM, a stage
// that fits at least once per consumer set
// consumer warps of the persistent kernel: rows up to 2048 wide, 12 where the group count divides 12, else the
// largest multiple of the count up to 16; rows up to 4096 wide need twice the registers per consumer, so 8 warps
// (group counts 1, 2, 4, 8).  0: the kernel does not take the shape.
constexpr int LNS_CONSUMERS_4K = 8;
static int layernorm_stream_consumers(int groups, int d) {
    if (groups < 1 || groups > LNS_CONSUMERS_WIDE) return 0;
    if (d > 4096) return 0;
    if (d > 2048) return LNS_CONSUMERS_4K % groups == 0 ? LNS_CONSUMERS_4K : 0;
    if (LNS_CONSUMERS % groups == 0) return LNS_CONSUMERS;
    return LNS_CONSUMERS_WIDE / groups * groups;
}

bool layernorm_stream_fits(const float *a, long long a_gstride, const float *y, int groups, int rows, int d,
                           int *stages_out) {
    const int n_consumers = layernorm_stream_consumers(groups, d);
    if (n_consumers == 0) return false;
    if ((d & 3) || (a_gstride & 3)) return false;
    if ((reinterpret_cast<uintptr_t>(a) & 15) || (reinterpret_cast<uintptr_t>(y) & 15)) return false;
    const int sms = sm_count() > 0 ? sm_count() : 148;
    if (rows < 8 * sms) return false;
    const int n_sets = n_consumers / groups;
    const long long stage_bytes = 4LL * d * (groups + (y ? 1 : 0));
    long long stages = (LNS_SMEM_BUDGET - 4LL * groups * d) / stage_bytes;   // gamma, beta sit behind the ring
    if (stages > LNS_MAX_STAGES) stages = LNS_MAX_STAGES;
    stages -= stages % n_sets;
    if (stages < 2) return false;
    *stages_out = static_cast<int>(stages);
    return true;
}

int launch_layernorm(const float *a, long long a_gstride, const float *y, const uint16_t *gamma,
                     const uint16_t *beta, int groups, int rows, int d, float eps, uint16_t *out,
                     cudaStream_t stream, const float *ysum, long long ysum_gstride, int ysum_groups,
                     uint32_t *status) {
    if (!a || !gamma || !out || groups < 1 || rows < 1 || d < 4 || (d & 3)) return KRAKEN_EINVAL;
    if (ysum && (y || ysum_groups < 1 || (ysum_gstride & 3))) return KRAKEN_EINVAL;
    int stages = 0;
    // the persistent kernel has bounded waits, so it needs a status word to report one that ran out
    if (status && !ysum && layernorm_stream_fits(a, a_gstride, y, groups, rows, d, &stages)) {
        const size_t smem = (size_t)stages * 4 * d * (groups + (y ? 1 : 0)) + (size_t)4 * groups * d;
        const int sms = sm_count() > 0 ? sm_count() : 148;
        const int n_consumers = layernorm_stream_consumers(groups, d);
        const bool wide = n_consumers > LNS_CONSUMERS;
        auto kern = d > 2048 ? layernorm_stream_kernel<32, LNS_CONSUMERS_4K>
                    : wide   ? (d <= 1024 ? layernorm_stream_kernel<8, LNS_CONSUMERS_WIDE>
                                          : layernorm_stream_kernel<16, LNS_CONSUMERS_WIDE>)
                             : (d <= 1024 ? layernorm_stream_kernel<8, LNS_CONSUMERS>
                                          : layernorm_stream_kernel<16, LNS_CONSUMERS>);
        static DeviceOnce configured[5];
        const int which = d > 2048 ? 4 : (wide ? 2 : 0) + (d <= 1024 ? 1 : 0);
        if (!configured[which].done()) {
            int rc = cuda_check(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     LNS_SMEM_BUDGET), "layernorm: shared memory opt-in");
            if (rc) return rc;
            configured[which].set();
        }
        const cudaError_t ce = launch_pdl(kern, dim3(sms), dim3((n_consumers + 1) * 32), smem, stream, a, a_gstride, y, gamma,
                                          beta, groups, rows, d, eps, out, stages, n_consumers, status);
        if (ce != cudaSuccess) return cuda_check(ce, "layernorm: launch");
        return cuda_check(cudaGetLastError(), "layernorm: launch");
    }
    const long long warps = (long long)groups * rows;
    // One CTA per row (layernorm_block_kernel) for rows of more than 2048 elements (a warp keeps 2048 in registers
    // and would go over the rest of the row three times) and for up to 24 rows per SM of more than 1024 elements.
    // Measured, 4 groups, us per launch, warp per row / CTA per row: 128 tokens d 2496 9.0 / 4.0, d 3120 11.3 / 4.5,
    // d 7424 29.1 / 6.3; 512 tokens d 2496 16.0 / 11.2; 2048 tokens d 2496 48.2 / 45.5, d 3120 61.2 / 50.3,
    // d 4992 121.7 / 66.7, d 7424 216.8 / 90.7; 8 groups d 3648 130.5 / 100.1; but d 2048 31.3 / 38.5 and 8 groups
    // d 1920 53.1 / 71.9.  KRAKEN_TUNE_LN_ROW_KERNEL = 1 / 2 forces the warp / the CTA per row.
    const int sms_b = sm_count() > 0 ? sm_count() : 148;
    const int force_b = tuning(KRAKEN_TUNE_LN_ROW_KERNEL);
    const bool block_auto = d > 2048 || (d > 1024 && warps <= 24LL * sms_b);
    const bool block_rows = !ysum && d <= 4 * LNB_THREADS * LNB_CACHE && (force_b ? force_b == 2 : block_auto);
    if (block_rows) {
        // a grid of resident CTAs that walk the rows: no second wave with a ragged tail
        static std::atomic<int> per_sm_of[MAX_DEVICES];
        const int dev = device_slot();
        if (dev < 0) return KRAKEN_ECUDA;
        int per_sm = per_sm_of[dev].load();
        if (per_sm == 0) {
            int n = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, layernorm_block_kernel, LNB_THREADS, 0) != cudaSuccess || n < 1) {
                cudaGetLastError();
                n = 4;
            }
            per_sm_of[dev].store(per_sm = n);
        }
        const long long resident = (long long)per_sm * sms_b;
        const long long ctas = warps < resident ? warps : resident;
        return cuda_check(launch_pdl(layernorm_block_kernel, dim3(static_cast<unsigned>(ctas)), dim3(LNB_THREADS), 0,
                                     stream, a, a_gstride, y, gamma, beta, groups, rows, d, eps, out),
                          "layernorm: launch");
    }
    const dim3 grid(static_cast<unsigned>((warps + ROW_WARPS - 1) / ROW_WARPS)), block(ROW_WARPS * 32);
    cudaError_t ce;
    if (ysum)
        ce = d <= 1024 ? launch_pdl(layernorm_kernel<8, true>, grid, block, 0, stream, a, a_gstride, y, ysum, ysum_gstride,
                                    ysum_groups, gamma, beta, groups, rows, d, eps, out)
                       : launch_pdl(layernorm_kernel<16, true>, grid, block, 0, stream, a, a_gstride, y, ysum, ysum_gstride,
                                    ysum_groups, gamma, beta, groups, rows, d, eps, out);
    else
        ce = d <= 1024 ? (grid.x > 3u * sms_b
                              ? launch_pdl(layernorm_kernel<8, false, true>, grid, block, 0, stream, a, a_gstride, y, ysum,
                                           ysum_gstride, ysum_groups, gamma, beta, groups, rows, d, eps, out)
                              : launch_pdl(layernorm_kernel<8, true>, grid, block, 0, stream, a, a_gstride, y, ysum,
                                           ysum_gstride, ysum_groups, gamma, beta, groups, rows, d, eps, out))
                       : launch_pdl(layernorm_kernel<16, false>, grid, block, 0, stream, a, a_gstride, y, ysum, ysum_gstride,
                                    ysum_groups, gamma, beta, groups, rows, d, eps, out);
    return cuda_check(ce, "layernorm: launch");
}

int launch_gather_concat(const float *x, long long x_gstride, int groups, int d, const int32_t *rows, int n_rows,
                         uint16_t *out, cudaStream_t stream) {
    if (!x || !out || groups < 1 || n_rows < 1 || (d & 3)) return KRAKEN_EINVAL;
    const long long warps = (long long)groups * n_rows;
    return cuda_check(launch_pdl(gather_concat_kernel, dim3(static_cast<unsigned>((warps + ROW_WARPS - 1) / ROW_WARPS)),
                                 dim3(ROW_WARPS * 32), 0, stream, x, x_gstride, groups, d, rows, n_rows, out),
                      "gather: launch");
}

int launch_gather_rows(const void *src, long long src_gstride_bytes, int groups, int row_bytes, const int32_t *rows,
                       int n_rows, void *dst, cudaStream_t stream) {
    if (!src || !dst || !rows || groups < 1 || n_rows < 1 || row_bytes < 16 || (row_bytes & 15) || (src_gstride_bytes & 15) ||
        (reinterpret_cast<uintptr_t>(src) & 15) || (reinterpret_cast<uintptr_t>(dst) & 15))
        return KRAKEN_EINVAL;
    const long long warps = (long long)groups * n_rows;
    return cuda_check(launch_pdl(gather_rows_kernel, dim3(static_cast<unsigned>((warps + ROW_WARPS - 1) / ROW_WARPS)),
                                 dim3(ROW_WARPS * 32), 0, stream, static_cast<const uint8_t *>(src), src_gstride_bytes,
                                 groups, row_bytes, rows, n_rows, static_cast<uint8_t *>(dst)),
                      "gather rows: launch");
}

int launch_sum_groups(const float *x, long long gstride, int groups, long long n, float *out, cudaStream_t stream) {
    if (!x || !out || groups < 1 || n < 4 || (n & 3) || (gstride & 3) || (reinterpret_cast<uintptr_t>(x) & 15) ||
        (reinterpret_cast<uintptr_t>(out) & 15))
        return KRAKEN_EINVAL;
    const long long n4 = n / 4;
    const int sms = sm_count() > 0 ? sm_count() : 148;
    long long blocks = (n4 + 255) / 256;
    if (blocks > 8LL * sms) blocks = 8LL * sms;
    return cuda_check(launch_pdl(sum_groups_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, stream, x, gstride,
                                 groups, n4, out),
                      "sum over groups: launch");
}

int launch_f32_to_bf16(const float *in, uint16_t *out, long long n, cudaStream_t stream) {
    if (n < 1) return KRAKEN_EINVAL;
    long long blocks = (n + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    f32_to_bf16_kernel<<<static_cast<unsigned>(blocks), 256, 0, stream>>>(in, out, n);
    return done();
}

}  // namespace kr
