// Host utilities: tensor-map encoding through the driver entry point, device queries, env flags.
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>

#include "internal.h"

#ifndef KRAKEN_F16
#define KRAKEN_F16 0
#endif

namespace kr {

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

int encode(CUtensorMap *map, const void *base, int rank, const uint64_t *dims, const uint64_t *strides_elems,
           const uint32_t *box) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return KRAKEN_ECUDA;
    cuuint64_t gdim[5], gstride[4];
    cuuint32_t bdim[5], estride[5];
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i];
        bdim[i] = box[i];
        estride[i] = 1;
    }
    for (int i = 0; i + 1 < rank; ++i) gstride[i] = strides_elems[i] * 2;  // bytes
    CUresult r = fn(map, (KRAKEN_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16), rank, const_cast<void *>(base), gdim, gstride, bdim,
                    estride, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? KRAKEN_OK : KRAKEN_ECUDA;
}

}  // namespace

int encode_tma_3d_bf16(CUtensorMap *map, const void *base, uint64_t dim0, uint64_t dim1, uint64_t dim2,
                       uint64_t stride1_elems, uint64_t stride2_elems, uint32_t box0, uint32_t box1) {
    const uint64_t dims[3] = {dim0, dim1, dim2};
    const uint64_t strides[2] = {stride1_elems, stride2_elems};
    const uint32_t box[3] = {box0, box1, 1};
    return encode(map, base, 3, dims, strides, box);
}

int encode_tma_4d_bf16(CUtensorMap *map, const void *base, const uint64_t dims[4], const uint64_t strides_elems[3],
                       const uint32_t box[4]) {
    return encode(map, base, 4, dims, strides_elems, box);
}

int device_slot() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return -1;
    return dev;
}

bool DeviceOnce::done() const {
    const int dev = device_slot();
    return dev >= 0 && flag[dev].load(std::memory_order_acquire) != 0;
}

void DeviceOnce::set() {
    const int dev = device_slot();
    if (dev >= 0) flag[dev].store(1, std::memory_order_release);
}

int sm_count() {
    static std::atomic<int> n[MAX_DEVICES];
    const int dev = device_slot();
    if (dev < 0) return 0;
    int v = n[dev].load(std::memory_order_relaxed);
    if (v <= 0) {
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        n[dev].store(v, std::memory_order_relaxed);
    }
    return v;
}

namespace {
std::atomic<int> g_tuning[KRAKEN_TUNE_COUNT];
}

int tuning(int key) { return key >= 0 && key < KRAKEN_TUNE_COUNT ? g_tuning[key].load(std::memory_order_relaxed) : 0; }

int set_tuning(int key, int value) {
    if (key < 0 || key >= KRAKEN_TUNE_COUNT || value < 0 || value > 3) return KRAKEN_EINVAL;
    g_tuning[key].store(value, std::memory_order_relaxed);
    return KRAKEN_OK;
}

static thread_local char g_last_error[256] = "";

int cuda_check(cudaError_t e, const char *where) {
    if (e == cudaSuccess) return KRAKEN_OK;
    snprintf(g_last_error, sizeof(g_last_error), "%s: %s", where, cudaGetErrorString(e));
    return KRAKEN_ECUDA;
}

const char *last_cuda_error() { return g_last_error; }

bool env_flag(const char *name) {
    const char *v = getenv(name);
    return v && *v && strcmp(v, "0") != 0;
}

}  // namespace kr
