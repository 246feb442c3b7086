// Decode-step attention for callers that cannot hand the library any scratch memory.
//
// Some hosts of this library never get to call cudaMalloc: an inference server that reserved the
// whole device for its own pool at start-up (a later allocation simply fails), a plugin whose
// contract passes it input and output pointers and nothing else, or a latency-critical loop in
// which the implicit device synchronisation of an allocation is not acceptable.  For them the
// split-KV partials live in the fixed array below, which is part of the loaded library image:
// every GPU that loads libkraken.so holds these bytes until the process exits.
#include <mutex>

#include "internal.h"

namespace {

// 2 Mi floats = 8 MiB: room for groups * batch * n_head * splits * (head_dim + 2) partial values.
constexpr size_t STATIC_PARTIAL_FLOATS = size_t(2) << 20;
static __device__ __align__(256) float g_decode_partials[STATIC_PARTIAL_FLOATS];

std::mutex g_setup_mutex;
float *g_partials_addr[kr::MAX_DEVICES] = {};  // device address of the array, per device ordinal

// In host code `g_decode_partials` is only a handle for the runtime, never a device address: the
// address a kernel can use must be asked for, once per device, with that device current.
// The array belongs to the current device, so the tensors of the call must live there too: `q` is
// looked up and a pointer into another device's memory is refused instead of being paired with
// this device's array.
int partials_address(const void *q, float **out) {
    const int dev = kr::device_slot();
    if (dev < 0) return KRAKEN_ECUDA;
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, q) != cudaSuccess) {
        cudaGetLastError();
        return KRAKEN_EINVAL;
    }
    if (attr.type == cudaMemoryTypeDevice && attr.device != dev) return KRAKEN_EINVAL;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_partials_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_decode_partials) != cudaSuccess || !p) return KRAKEN_ECUDA;
        g_partials_addr[dev] = static_cast<float *>(p);
    }
    *out = g_partials_addr[dev];
    return KRAKEN_OK;
}

}  // namespace

extern "C" int kraken_op_decode_attention_static(const void *q, int64_t q_gstride, const void *k_cache,
                                                 const void *v_cache, int64_t cache_gstride, int64_t cache_bstride,
                                                 int32_t groups, int32_t batch, int32_t n_keys, int32_t n_head,
                                                 int32_t head_dim, int32_t max_pos, int32_t splits, void *out,
                                                 int64_t out_gstride, void *stream) {
    using namespace kr;
    if (groups < 1 || batch < 1 || n_head < 1 || n_keys < 1) return KRAKEN_EINVAL;
    if (!q || !k_cache || !v_cache || !out) return KRAKEN_EINVAL;
    if (!decode_head_dim_ok(head_dim)) return KRAKEN_EUNSUPPORTED;
    if (splits == 0) splits = decode_attention_splits(groups, batch, n_head, n_keys);
    if (splits < 1 || splits > DECODE_MAX_SPLITS) return KRAKEN_EINVAL;
    const size_t need = decode_attention_partial_bytes(groups, batch, n_head, head_dim, splits);
    if (splits > 1 && need > STATIC_PARTIAL_FLOATS * sizeof(float)) return KRAKEN_ECAPACITY;
    float *partials = nullptr;
    int rc = partials_address(q, &partials);
    if (rc) return rc;
    DecodeAttnParams p;
    p.q = static_cast<const uint16_t *>(q);
    p.q_gstride = q_gstride;
    p.k_cache = static_cast<const uint16_t *>(k_cache);
    p.v_cache = static_cast<const uint16_t *>(v_cache);
    p.cache_gstride = cache_gstride;
    p.cache_bstride = cache_bstride;
    p.groups = groups;
    p.batch = batch;
    p.n_keys = n_keys;
    p.n_head = n_head;
    p.head_dim = head_dim;
    p.max_pos = max_pos;
    p.pos_dev = nullptr;
    p.splits = splits;
    p.partials = partials;
    p.out = static_cast<uint16_t *>(out);
    p.out_gstride = out_gstride;
    return launch_attention_decode(p, static_cast<cudaStream_t>(stream));
}

extern "C" size_t kraken_decode_attention_static_capacity(void) { return STATIC_PARTIAL_FLOATS * sizeof(float); }
