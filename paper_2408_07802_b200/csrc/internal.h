// Declarations shared by the translation units of the library (host side).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/kraken.h"

namespace kr {

// Epilogue description handed to the GEMM kernels (device pointers, strides in elements).
struct EpiParams {
    int kind;  // kraken_epilogue
    const uint16_t *bias;
    long long bias_gstride;
    float *out_f32;
    long long out_f32_gstride;
    int ld_out_f32;
    uint16_t *out_bf16;
    long long out_bf16_gstride;
    int ld_out_bf16;
    const float *resid;
    long long resid_gstride;
    int ld_resid;
    float *sum;
    int ld_sum;
    uint16_t *k_cache, *v_cache;
    long long cache_gstride;
    int seqlen, pos0, n_head, head_dim, max_pos, d_model;
    int n_kv_head;  // key/value heads (grouped-query attention); the k and v parts are n_kv_head * head_dim wide
    int gelu_tanh;
    // when set, the first position of sequence b is pos0_dev[b] in device memory (replayable decode graph,
    // sequences of different lengths)
    const int *pos0_dev;
    // packed (ragged) prefill: row r belongs to sequence row_seq[r] at position row_pos[r]
    const int *row_seq, *row_pos;
    // LayerNorm of the finished rows in the same kernel (RESID_F32 and RESID_SUM only; ln_out != NULL turns it on):
    //   ln_out[g] = LN(out_f32[g] + ln_y; gamma[g], beta[g])   over the whole row of n_out columns.
    // A row is spread over the N tiles of its row block, i.e. over several CTAs, so every epilogue warp leaves
    // the (mean, M2, count) of its part of each row in ln_parts, counts itself in ln_cnt, waits (bounded) for the
    // other parts of its 32 rows and then normalises the values it kept in tensor memory.
    uint16_t *ln_out;
    long long ln_out_gstride;
    int ln_ld_out;
    const uint16_t *ln_gamma, *ln_beta;   // [G][n_out]; beta may be NULL
    long long ln_gb_gstride;
    const float *ln_y;                    // [M, n_out] added before the statistics, or NULL
    int ln_ld_y;
    float ln_eps;
    float4 *ln_parts;                     // [G][M][ln_n_parts]
    uint32_t *ln_cnt;                     // [G][ceil(M / 32)][2]: arrivals, departures; zero between launches
    int ln_n_parts;                       // 2 * N tiles, filled in by the launcher
};

// Scratch of the fused LayerNorm for a launch of `groups` x `m` rows whose rows are `n_out` wide and cut into
// tiles of `bn` columns (GEMM_TILE_PAIR: 256): bytes of the parts array and of the counters.
size_t gemm_ln_parts_bytes(int groups, int m, int n_out, int bn);
size_t gemm_ln_cnt_bytes(int groups, int m);

struct GemmShape {
    int groups, m, n_out, k;
};

// Host-resolved driver entry point for tensor-map encoding; returns KRAKEN_ECUDA if unavailable.
int encode_tma_3d_bf16(CUtensorMap *map, const void *base, uint64_t dim0, uint64_t dim1, uint64_t dim2,
                       uint64_t stride1_elems, uint64_t stride2_elems, uint32_t box0, uint32_t box1);
int encode_tma_4d_bf16(CUtensorMap *map, const void *base, const uint64_t dims[4], const uint64_t strides_elems[3],
                       const uint32_t box[4]);

// Launch set-up (shared-memory opt-ins, occupancy queries, the SM count) belongs to a device, not to the
// process: a host may drive several GPUs.  State is kept per device ordinal of the current device.
constexpr int MAX_DEVICES = 64;
int device_slot();   // ordinal of the current device, -1 if it cannot be had or is out of range
struct DeviceOnce {  // zero-initialised static: "this set-up has been done on the current device"
    std::atomic<unsigned char> flag[MAX_DEVICES];
    bool done() const;
    void set();
};
int sm_count();      // of the current device; 0 on failure

// Process-wide kernel choices for tests and measurements (kraken_tuning_set); 0 = the library's own choice.
int tuning(int key);
int set_tuning(int key, int value);

// Tensor-core grouped GEMM.  tmA / tmB may be NULL: they are then encoded from the operands.
// b_g0: index of the first group along the outermost dimension of a caller-made tmB (a map
// that spans the weights of every layer).
struct GemmOperands {
    const void *a;
    long long a_gstride;
    int lda;
    const void *w;
    long long w_gstride;
    int ldw;
    bool w_static = false;   // W is not written by the kernel before this one in the stream (model weights)
};
int launch_gemm_tc(const GemmOperands &op, const GemmShape &shape, const EpiParams &epi, const CUtensorMap *tmA,
                   const CUtensorMap *tmB, int b_g0, int bn_hint, uint32_t *d_status, cudaStream_t stream);
// Picks the N tile for a shape: 64, 128 or 256 (one CTA per 128-row tile), or GEMM_TILE_PAIR
// (two CTAs of a cluster share a 256 x 256 tile).
constexpr int GEMM_TILE_PAIR = 512;
int gemm_pick_bn(const GemmShape &shape);
int gemm_encode_a(CUtensorMap *map, const GemmOperands &op, const GemmShape &shape);
int gemm_encode_b(CUtensorMap *map, const GemmOperands &op, const GemmShape &shape, int bn);

// Weight-streaming GEMM for M <= 32 rows (decode, last-position tail); every epilogue except RESID_SUM.
int launch_gemm_skinny(const GemmOperands &op, const GemmShape &shape, const EpiParams &epi, cudaStream_t stream);
constexpr int SKINNY_MAX_ROWS = 32;

int launch_embed(const int32_t *ids, int n_tokens, int seqlen, int pos0, const uint16_t *wte, const uint16_t *wpe,
                 int d, int vocab, float *out, uint32_t *status, cudaStream_t stream, const int *pos0_dev = nullptr,
                 const int *row_pos = nullptr);
// y: [rows, d] added before normalisation (or NULL); alternatively ysum: `ysum_groups` tensors
// [rows, d], ysum_gstride apart, whose sum is added.
int launch_layernorm(const float *a, long long a_gstride, const float *y, const uint16_t *gamma,
                     const uint16_t *beta, int groups, int rows, int d, float eps, uint16_t *out,
                     cudaStream_t stream, const float *ysum = nullptr, long long ysum_gstride = 0,
                     int ysum_groups = 0, uint32_t *status = nullptr);
// out[i] = sum over groups of x[g * gstride + i], ascending g; n elements (a multiple of 4), 16-byte aligned
int launch_sum_groups(const float *x, long long gstride, int groups, long long n, float *out, cudaStream_t stream);
// rows of N fp32 branch outputs -> bf16 branch-major concatenation [n_rows, N*d]; rows picked by index list
// (device int32, NULL = identity).
int launch_gather_concat(const float *x, long long x_gstride, int groups, int d, const int32_t *rows, int n_rows,
                         uint16_t *out, cudaStream_t stream);
int launch_f32_to_bf16(const float *in, uint16_t *out, long long n, cudaStream_t stream);
// dst[g][i][:] = src[g][rows[i]][:]; rows of row_bytes bytes (a multiple of 16); rows: device int32 [n_rows]
int launch_gather_rows(const void *src, long long src_gstride_bytes, int groups, int row_bytes, const int32_t *rows,
                       int n_rows, void *dst, cudaStream_t stream);

struct AttnParams {
    const uint16_t *q;
    long long q_gstride;
    const uint16_t *k_cache, *v_cache;
    long long cache_gstride, cache_bstride;
    int groups, batch, seqlen, pos0, n_head, head_dim, max_pos;
    uint16_t *out;
    long long out_gstride;
    int n_kv_head = 0;  // key/value heads in the cache (0 = n_head); query head h reads head h / (n_head / n_kv_head)
};
// tcgen05 / TMEM attention for tiles of 128 queries x 128 keys; tensor maps may be NULL (encoded per call).
bool attention_tc_supported(const AttnParams &p);
int attention_tc_encode(const AttnParams &p, CUtensorMap *tmQ, CUtensorMap *tmK, CUtensorMap *tmV);
int launch_attention_tc(const AttnParams &p, const CUtensorMap *tmQ, const CUtensorMap *tmK, const CUtensorMap *tmV,
                        uint32_t *d_status, cudaStream_t stream);

// Decode-step attention (one query row per sequence and head) with split-KV partials in scratch.
constexpr int DECODE_MAX_SPLITS = 32;
struct DecodeAttnParams {
    const uint16_t *q;  // [G][batch, d]
    long long q_gstride;
    const uint16_t *k_cache, *v_cache;
    long long cache_gstride, cache_bstride;
    int groups, batch, n_keys, n_head, head_dim, max_pos;
    int n_kv_head = 0;   // key/value heads in the cache (0 = n_head)
    const int *pos_dev;  // when set, sequence b has n_keys = pos_dev[b] + 1 (replayable decode graph, ragged batches)
    int splits;
    float *partials;  // [G*batch*n_head][splits][head_dim + 2] fp32 (max, sum, output); unused when splits == 1
    uint16_t *out;    // [G][batch, d]
    long long out_gstride;
};
inline bool decode_head_dim_ok(int hd) { return hd == 64 || hd == 72 || hd == 96 || hd == 104 || hd == 128; }
int decode_attention_splits(int groups, int batch, int n_head, int n_keys);
// whether the query heads of a key/value head are served together by the tensor-core tile kernel (then the
// number of CTA streams, which the split count should be chosen for, is the number of key/value heads)
bool decode_gqa_tile(int n_head, int n_kv_head);
size_t decode_attention_partial_bytes(int groups, int batch, int n_head, int head_dim, int splits);
int launch_attention_decode(const DecodeAttnParams &p, cudaStream_t stream);

// Launch with programmatic stream serialisation (see pdl_wait / pdl_trigger in ptx.cuh): hides the
// launch latency between the many short kernels of a decode step.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

bool env_flag(const char *name);
// Records the text of a failed CUDA call (per thread) and maps it to KRAKEN_ECUDA.
int cuda_check(cudaError_t e, const char *where);
const char *last_cuda_error();

}  // namespace kr
