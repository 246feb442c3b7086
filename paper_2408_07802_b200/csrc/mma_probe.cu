// Issue-rate probe for the tensor-core products of the attention kernel: how many SM clock cycles one
// `tcgen05.mma` of M 128, K 16 costs when ONE thread per SM issues them back to back, and when two threads in
// different warps do, for the operand forms the attention kernel uses (S = Q K^T: both operands in shared
// memory; O += P V: A from tensor memory, V MN-major in shared memory) and for N = 64 / 128 / 256.
// A measurement tool beside the model kernels (like the wait probe): it explains why a one-issuer attention
// step cannot run at the tensor rate while the GEMM kernels' N = 256 products do.  Operands are zeros in shared
// memory and whatever tensor memory holds; the timing does not depend on the data.  All waits are bounded.
#include "internal.h"
#include "ptx.cuh"

namespace kr {

namespace {

constexpr int PROBE_THREADS = 96;                 // warp 0: set-up; warps 1 and 2: the issuing threads
constexpr int PROBE_OPERAND_BYTES = 160 * 1024;   // Q 2 x 32 KB, K up to 64 KB (N 256), V 32 KB
constexpr int PROBE_SMEM_BYTES = PROBE_OPERAND_BYTES + 1024 + 256;

__device__ __forceinline__ uint64_t desc_sw128_mnmajor(uint32_t smem_addr, uint32_t lbo_bytes) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= static_cast<uint64_t>(1024 >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(2) << 61;
    return d;
}

// form: 0 = Q K^T (N 128), 1 = P V, 2 = 8 Q K^T then 8 P V alternating (the attention kernel's pattern),
//       3 = form 2 with a commit after every 8, 4 = form 3 with a barrier wait that succeeds at once after every 8,
//       5 = Q K^T with N 64, 6 = Q K^T with N 256
__global__ void __launch_bounds__(PROBE_THREADS, 1)
mma_probe_kernel(int form, int issuers, int iters, long long *cycles, uint32_t *status) {
    extern __shared__ uint8_t probe_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(probe_raw) + 1023) & ~uintptr_t(1023));
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + PROBE_OPERAND_BYTES);   // 0, 1: commits nobody waits for;
    uint32_t *slot = reinterpret_cast<uint32_t *>(bars + 8);                      // 2: already complete; 3, 4: the end
    volatile uint32_t *abort_flag = slot + 1;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < PROBE_OPERAND_BYTES / 16; i += PROBE_THREADS)
        reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
    if (threadIdx.x == 0) {
        for (int i = 0; i < 8; ++i) mbar_init(bars + i, 1);
        *abort_flag = 0;
        fence_barrier_init();
        mbar_arrive(bars + 2);   // its first phase is complete from the start
    }
    if (warp == 1) {
        tmem_alloc(slot, 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = *slot;
    const int me = warp - 1;      // issuing thread 0 or 1
    if ((warp == 1 || (warp == 2 && issuers == 2)) && lane == 0) {
        const uint32_t q = smem_u32(smem), k = smem_u32(smem + 65536), v = smem_u32(smem + 131072);
        const uint32_t idesc_128 = umma_idesc_h16(128, 128), idesc_64 = umma_idesc_h16(128, 64),
                       idesc_256 = umma_idesc_h16(128, 256), idesc_pv = umma_idesc_h16(128, 128) | (1u << 16);
        bool ok = true;
        const long long t0 = clock64();
        for (int it = 0; ok && it < iters; ++it) {
            // one issuing thread alternates between the two query tiles' accumulators per block of 8, two issuing
            // threads keep to their own
            const int w = issuers == 2 ? me : (it & 1);
            if (form == 0 || form == 2 || form == 3 || form == 4) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t off = (ks >> 2) * 16384 + (ks & 3) * 32;
                    umma_bf16_ss(tm + w * 128, umma_desc_sw128_kmajor(q + w * 32768 + off), umma_desc_sw128_kmajor(k + off),
                                 idesc_128, ks != 0 ? 1u : 0u);
                }
                if (form >= 3) umma_commit(bars + me);
                if (form == 4) {
                    ok = mbar_wait(bars + 2, 0, abort_flag);
                    tc_fence_after_sync();
                }
            }
            if (form == 5) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t off = (ks >> 2) * 16384 + (ks & 3) * 32;
                    umma_bf16_ss(tm + w * 128, umma_desc_sw128_kmajor(q + w * 32768 + off), umma_desc_sw128_kmajor(k + off),
                                 idesc_64, ks != 0 ? 1u : 0u);
                }
            }
            if (form == 6) {   // 256 columns: the two threads of a two-issuer run take columns 0..255 and 256..511
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t off = (ks & 3) * 32;
                    umma_bf16_ss(tm + (issuers == 2 ? me * 256 : 0), umma_desc_sw128_kmajor(q + w * 32768 + (ks >> 2) * 16384 + off),
                                 umma_desc_sw128_kmajor(k + (ks >> 2) * 32768 + off), idesc_256, ks != 0 ? 1u : 0u);
                }
            }
            if (form >= 1 && form <= 4) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    umma_bf16_ts(tm + 256 + w * 128, tm + w * 128 + ks * 8, desc_sw128_mnmajor(v + ks * 2048, 16384), idesc_pv, 1u);
                if (form >= 3) umma_commit(bars + me);
                if (form == 4) {
                    ok = mbar_wait(bars + 2, 0, abort_flag);
                    tc_fence_after_sync();
                }
            }
        }
        // every product issued by this thread has finished when its last commit arrives
        umma_commit(bars + 3 + me);
        if (!mbar_wait(bars + 3 + me, 0, abort_flag)) ok = false;
        const long long t1 = clock64();
        if (me == 0) cycles[blockIdx.x] = ok ? t1 - t0 : -1;
    }
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
        if (threadIdx.x == 0 && status) atomicOr(status, STATUS_WAIT_LIMIT);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tm, 512);
}

}  // namespace

}  // namespace kr

extern "C" int kraken_test_mma_issue_rate(int32_t form, int32_t issuers, int32_t iters, int64_t *d_cycles,
                                          int32_t n_ctas, int32_t *products_per_iter, uint32_t *d_status, void *stream) {
    using namespace kr;
    if (form < 0 || form > 6 || (issuers != 1 && issuers != 2) || iters < 1 || iters > 100000 || !d_cycles ||
        n_ctas < 1 || n_ctas > 1024)
        return KRAKEN_EINVAL;
    static DeviceOnce configured;
    if (!configured.done()) {
        int rc = cuda_check(cudaFuncSetAttribute(mma_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 PROBE_SMEM_BYTES), "mma probe: shared memory opt-in");
        if (rc) return rc;
        configured.set();
    }
    if (products_per_iter) *products_per_iter = (form >= 2 && form <= 4) ? 16 : 8;
    mma_probe_kernel<<<n_ctas, PROBE_THREADS, PROBE_SMEM_BYTES, static_cast<cudaStream_t>(stream)>>>(
        form, issuers, iters, reinterpret_cast<long long *>(d_cycles), d_status);
    return cuda_check(cudaGetLastError(), "mma probe: launch");
}
