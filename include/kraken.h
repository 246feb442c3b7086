/*
 * kraken.h - C ABI of the single-GPU Kraken prefill / decode library (sm_100a).
 *
 * A Kraken model (Prabhakar et al., "Kraken: Inherently Parallel Transformers For
 * Efficient Multi-Device Inference") has L layers of N independent sub-layers
 * ("branches").  Algorithm 1 defines one sub-layer:
 *     res = x;  y = AllReduce(x);  x = LN(x);  x = res + MHA(x);
 *     res = x;  x = LN(x + y);     out = res + FFN(x)
 * with the AllReduce an element-wise sum over the N sub-layer inputs (identity in the
 * first layer), one shared token+position embedding, and a final linear map W_concat
 * over the concatenated N outputs before the tied unembedding (Sec. 3.1).  This library
 * runs all N branches on ONE device: the branches are the group dimension of grouped
 * GEMMs and the AllReduce is a sum inside the down-projection's epilogue.
 *
 * Conventions for every call
 *   - "device" pointers are CUDA device memory of the current device; "host" pointers
 *     are ordinary (preferably pinned) host memory.  The library never allocates device
 *     memory: weights, KV cache, scratch, tokens and logits are caller-owned.
 *   - 16-bit tensors ("bf16" below) are raw 16-bit patterns, row-major, innermost dimension
 *     contiguous.  The library comes as two images of the same ABI: libkraken.so stores weights,
 *     activations and the KV cache as bfloat16, libkraken_f16.so as IEEE half (the precision of the
 *     paper's engines, Sec. 4.2); wherever this header says bf16 the second image means half.
 *     kraken_storage_dtype() tells which one is loaded.  Accumulation, the residual stream and the
 *     logits are fp32 in both.
 *   - Calls only enqueue work on the given stream (a cudaStream_t passed as void*; NULL
 *     is the legacy default stream) unless stated otherwise.
 *   - Every call returns 0 or a negative kraken_status.  Nothing aborts, throws across
 *     the boundary or traps on the device.
 */
#ifndef KRAKEN_H_
#define KRAKEN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum kraken_status {
    KRAKEN_OK = 0,
    KRAKEN_EINVAL = -1,       /* null / non-positive / inconsistent argument                  */
    KRAKEN_EUNSUPPORTED = -2, /* shape outside what the kernels support (see kraken_create)   */
    KRAKEN_ECAPACITY = -3,    /* batch, sequence or buffer larger than the handle was sized for */
    KRAKEN_ESTATE = -4,       /* call order violated (decode before prefill, batch changed)   */
    KRAKEN_ECUDA = -5         /* a CUDA runtime / driver call failed                          */
} kraken_status;

/* Model hyper-parameters and capacity (the analogue of an inference engine's build-time maxima). */
typedef struct kraken_config {
    int32_t n_branch;  /* N: sub-layers per layer, the paper's degree of parallelism (Sec. 3.1) */
    int32_t n_layer;   /* L                                                                   */
    int32_t d_model;   /* d: width of ONE sub-layer                                           */
    int32_t n_head;    /* attention heads per sub-layer (Table 3 caption); head_dim = d / n_head */
    int32_t d_ff;      /* FFN hidden width (4d standard, 2d for parameter parity; Sec. 3.2)   */
    int32_t vocab;     /* V                                                                   */
    int32_t max_pos;   /* rows of the position table = KV capacity per sequence               */
    int32_t max_batch; /* sequences per call                                                  */
    float ln_eps;      /* LayerNorm epsilon (1e-5)                                            */
    int32_t gelu_tanh; /* 0: GELU by erf (default), 1: tanh approximation                     */
    int32_t final_ln;  /* 1: LayerNorm between W_concat and the unembedding (default), 0: none */
    int32_t n_kv_head; /* key/value heads per sub-layer: 0 or n_head = multi-head attention; a divisor of
                          n_head = grouped-query attention, 1 = multi-query attention (the KV-cache
                          mitigation of Sec. 4.2): query head h reads key/value head h / (n_head / n_kv_head) */
    int32_t no_combine;/* 1: no cross-branch term (y = 0 in every layer).  With n_branch = 1 the layers are those
                          of the standard pre-LayerNorm Transformer the paper compares against (Sec. 4.2), on
                          the same kernels; 0 (default): Algorithm 1 */
    int32_t parallel_ffn; /* 1: the FFN reads the first LayerNorm's output, in parallel with attention:
                          out = x + MHA(LN(x)) + FFN(LN(x)) - the "Parallel Attention + FeedForward"
                          comparison architecture of Sec. 4.2; ln2 weights are then unused and there is no y */
    int32_t reserved[2];
} kraken_config;

/* Device pointers to bf16 weights, row-major [out_features, in_features]; BORROWED until
 * kraken_destroy.  Any bias or LayerNorm-beta pointer may be NULL (= zeros).
 * w_qkv rows 0..d-1 produce Q, the next kvd = n_kv_head*hd rows K, the last kvd rows V (kvd = d for
 * multi-head attention); head h owns rows h*hd..(h+1)*hd-1 of each part.
 * w_concat input index n*d + j is feature j of branch n (branch-major concatenation). */
typedef struct kraken_weights {
    const void *wte;                /* [V, d] token embedding, also the unembedding (tied) */
    const void *wpe;                /* [max_pos, d] learned positions                     */
    const void *ln1_g, *ln1_b;      /* [L][N][d]                                          */
    const void *w_qkv, *b_qkv;      /* [L][N][d+2kvd][d], [L][N][d+2kvd]                  */
    const void *w_proj, *b_proj;    /* [L][N][d][d],  [L][N][d]                           */
    const void *ln2_g, *ln2_b;      /* [L][N][d]                                          */
    const void *w_up, *b_up;        /* [L][N][F][d],  [L][N][F]                           */
    const void *w_down, *b_down;    /* [L][N][d][F],  [L][N][d]                           */
    const void *w_concat, *b_concat;/* [d][N*d], [d]                                      */
    const void *lnf_g, *lnf_b;      /* [d]; ignored when final_ln == 0                    */
} kraken_weights;

typedef struct kraken_handle kraken_handle;

/* Bytes of KV cache and scratch a handle of this configuration needs.  Pure host
 * arithmetic, usable without a GPU.  KV layout: [L][N][2 (K,V)][max_batch][n_kv_head][max_pos][head_dim] bf16.
 * Errors: EINVAL (null, non-positive field, d % n_head != 0), EUNSUPPORTED (see kraken_create). */
int kraken_query_sizes(const kraken_config *cfg, size_t *kv_bytes, size_t *scratch_bytes);

/* Build a handle: validates the configuration, records the borrowed weight pointers and
 * the caller's KV and scratch buffers (device, 256-byte aligned, at least the queried
 * sizes), encodes the TMA descriptors of the weights.  Host work only.
 * Supported shapes: head_dim in {64, 72, 96, 104, 128}; d_model and d_ff multiples of 8.
 * Errors: EINVAL, EUNSUPPORTED, ECAPACITY (undersized buffers), ECUDA. */
int kraken_create(const kraken_config *cfg, const kraken_weights *weights, void *d_kv, size_t kv_bytes,
                  void *d_scratch, size_t scratch_bytes, kraken_handle **out);

/* Prefill (Sec. 2.1: the step that produces the first token and the KV cache).
 * d_tokens: device int32 [batch, seqlen] row-major, all sequences the same length;
 * d_logits: device fp32 [batch, V], logits of the LAST position of each sequence.
 * Fills the KV cache rows 0..seqlen-1 of sequences 0..batch-1 and sets the handle's
 * length to seqlen.  Token ids outside [0, V) are read as 0 and raise status bit 0.
 * Only the last position's logits are returned, so past its Q_K_V product (whose K and V rows the cache needs
 * for every position) the LAST layer runs for the last position of every sequence only: its queries attend over
 * the cache like a decode step, and the output projection, the second LayerNorm and the FFN see batch rows.
 * The results are those of Algorithm 1 for these rows; the work for the other rows of that layer is not done
 * (kraken_logits_rows does it when asked for them).  kraken_prefill_packed does the same.
 * Errors: EINVAL, ECAPACITY (batch > max_batch, seqlen > max_pos), ECUDA. */
int kraken_prefill(kraken_handle *h, const int32_t *d_tokens, int32_t batch, int32_t seqlen,
                   float *d_logits, void *stream);

/* Same with HOST buffers: copies the tokens to the device, runs the prefill, copies the
 * logits back and synchronises the stream before returning.  h_tokens [batch, seqlen],
 * h_logits [batch, V]. */
int kraken_prefill_host(kraken_handle *h, const int32_t *h_tokens, int32_t batch, int32_t seqlen,
                        float *h_logits, void *stream);

/* Prefill of a batch whose sequences have different lengths, without padding ("packed" input): d_tokens
 * holds the sequences back to back (device int32, sum of the lengths), h_seq_lens their lengths (HOST,
 * read before the call returns), d_logits device fp32 [batch, V] = the logits of every sequence's last
 * position.  Sequence b fills rows 0 .. len_b - 1 of its own slice of the KV cache (kraken_kv_view), and the
 * decode steps that follow continue every sequence at its own position.  kraken_logits_rows then counts
 * rows in the packed order.  Errors: EINVAL (a length < 1), ECAPACITY (batch > max_batch, a length >
 * max_pos). */
int kraken_prefill_packed(kraken_handle *h, const int32_t *d_tokens, const int32_t *h_seq_lens, int32_t batch,
                          float *d_logits, void *stream);

/* ------------------------------------------------------------------------------------------
 * Branch-parallel deployment (the paper's own: each device holds some of the N branches of every
 * layer, Fig. 3 and App. A.2).  A handle created with the LOCAL branches' weights (n_branch = the
 * number held here, w_concat = the columns of W_concat that multiply those branches, b_concat only
 * on one device) is driven in pieces, so that the caller can sum the layer outputs over all devices
 * (the AllReduce of Algorithm 1) while the next layer's attention half is already running - the
 * overlap the paper builds its latency claim on (Sec. 3.1):
 *
 *   kraken_stage_begin(tokens)                      shared embedding x0 (identical on every device)
 *   for layer l = 0 .. L-1:
 *       kraken_stage_attention(l)                   LN1, qkv, attention, proj + residual
 *       kraken_stage_ffn(l, y)                      LN2(. + y), up, GELU, down + residual; then the sum
 *                                                   of this device's layer outputs is in d_local_sum
 *           y = x0 for l = 0, else the sum over ALL devices of the d_local_sum of layer l-1
 *           (the caller's all-reduce; it must be complete before kraken_stage_ffn(l) is enqueued
 *           and may run while kraken_stage_attention(l) does)
 *   kraken_stage_concat(z)                          this device's part of W_concat at the last positions
 *   (caller: sum z over all devices)
 *   kraken_stage_head(z, logits)                    final LayerNorm, unembedding; the prefill is then
 *                                                   complete (cur_len = seqlen) and kraken_kv_view valid
 *
 * d_y, d_z: device fp32 [batch*seqlen, d] and [batch, d]; kraken_stage_buffers returns the device
 * addresses of x0 and of the local-sum buffer ([batch*seqlen, d] fp32, overwritten by every
 * kraken_stage_ffn).  Calls out of order return ESTATE.  With one device holding all branches the
 * sequence computes exactly what kraken_prefill computes.  A decode step is driven the same way after
 * kraken_stage_begin_decode(tokens [batch]) (one new token per sequence; d_y and the local sum are then
 * [batch, d]); its kraken_stage_head advances every sequence by one position.
 * ------------------------------------------------------------------------------------------ */
int kraken_stage_begin(kraken_handle *h, const int32_t *d_tokens, int32_t batch, int32_t seqlen, void *stream);
int kraken_stage_begin_decode(kraken_handle *h, const int32_t *d_tokens, int32_t batch, void *stream);
int kraken_stage_attention(kraken_handle *h, int32_t layer, void *stream);
int kraken_stage_ffn(kraken_handle *h, int32_t layer, const float *d_y, void *stream);
int kraken_stage_buffers(kraken_handle *h, float **d_x0, float **d_local_sum);
int kraken_stage_concat(kraken_handle *h, float *d_z, void *stream);
int kraken_stage_head(kraken_handle *h, const float *d_z, float *d_logits, void *stream);

/* Current length of every cached sequence (host array of `batch` entries; kraken_cur_len is their maximum).
 * ESTATE when batch differs from the cached batch. */
int kraken_seq_lens(kraken_handle *h, int32_t *h_seq_lens, int32_t batch);

/* Prefill that returns the logits of EVERY position: d_logits device fp32 [batch, seqlen, V].
 * Same cache side effects as kraken_prefill.  Meant for tests and evaluation. */
int kraken_prefill_all_logits(kraken_handle *h, const int32_t *d_tokens, int32_t batch, int32_t seqlen,
                              float *d_logits, void *stream);

/* Logits of chosen token rows of the most recent prefill (its last-layer outputs stay in
 * scratch until the next call that runs the model; after a prefill that ran its last layer for the last
 * positions only, this call first runs that layer on every row, from the inputs the prefill left in scratch).
 * h_rows: HOST int32 [n_rows], row = b*seqlen + t;
 * d_logits: device fp32 [n_rows, V].  Errors: EINVAL, ESTATE (no prefill yet), ECAPACITY (n_rows
 * larger than max_batch * max_pos). */
int kraken_logits_rows(kraken_handle *h, const int32_t *h_rows, int32_t n_rows, float *d_logits, void *stream);

/* One decode step (Sec. 2.1): one new token per sequence at position cur_len, attending to
 * cache rows 0..cur_len (the new one included); appends K,V; cur_len += 1.
 * d_tokens device int32 [batch]; d_logits device fp32 [batch, V].
 * Errors: ESTATE (no prefill, or batch differs from the prefill's), ECAPACITY (cur_len == max_pos). */
int kraken_decode_step(kraken_handle *h, const int32_t *d_tokens, int32_t batch, float *d_logits, void *stream);

/* Same with HOST buffers (h_tokens [batch], h_logits [batch, V]); synchronises the stream. */
int kraken_decode_step_host(kraken_handle *h, const int32_t *h_tokens, int32_t batch, float *h_logits, void *stream);

/* Where the cache of (layer, branch, which: 0 = K, 1 = V) lives: base device pointer and
 * strides in ELEMENTS for (batch, head, position, dim). */
int kraken_kv_view(kraken_handle *h, int32_t layer, int32_t branch, int32_t which, const void **ptr,
                   int64_t strides[4]);

/* Synchronises the stream of the last call and reports the device status word:
 * bit 0 = a token id was out of range, bit 1 = a bounded wait inside a kernel gave up. */
int kraken_device_status(kraken_handle *h, uint32_t *flags);

/* Current sequence length held in the cache (0 before any prefill). */
int kraken_cur_len(kraken_handle *h, int32_t *cur_len);

/* Launch accounting and per-kernel timing.  Every call that runs the model counts its kernel
 * launches per category; with profiling enabled each launch is also bracketed by CUDA events on
 * the call's stream.  kraken_profile_read synchronises that stream, returns the accumulated
 * device milliseconds (0 when profiling was off) and launch counts since the last read, and
 * resets them.  ms, launches: HOST arrays of KRAKEN_PROF_COUNT entries. */
typedef enum kraken_prof_category {
    KRAKEN_PROF_EMBED = 0,
    KRAKEN_PROF_LAYERNORM = 1,
    KRAKEN_PROF_GEMM_QKV = 2,
    KRAKEN_PROF_ATTENTION = 3,
    KRAKEN_PROF_GEMM_PROJ = 4,
    KRAKEN_PROF_GEMM_UP = 5,
    KRAKEN_PROF_GEMM_DOWN = 6,
    KRAKEN_PROF_TAIL = 7,      /* row gather, W_concat, final LayerNorm, unembedding */
    KRAKEN_PROF_COUNT = 8
} kraken_prof_category;
int kraken_profile_enable(kraken_handle *h, int32_t on);
int kraken_profile_read(kraken_handle *h, double *ms, int64_t *launches);

/* Forget the cached sequences (cur_len = 0, status word cleared). */
int kraken_reset(kraken_handle *h);
void kraken_destroy(kraken_handle *h);
const char *kraken_strerror(int status);
/* Text of the most recent CUDA failure behind a KRAKEN_ECUDA on the calling thread ("" if none). */
const char *kraken_last_cuda_error(void);
/* 16-bit storage type this image was built for: 0 = bfloat16, 1 = IEEE half. */
int kraken_storage_dtype(void);

/* Hooks for tests and measurements (not part of the model's arithmetic).  Where the library has two kernels
 * for one step that give the same result and picks by shape, a test can force either one, process-wide:
 * value 0 restores the library's own choice.  Set a value before the handle that should see it is created (a handle
 * may replay a launch sequence it recorded earlier).  Nothing on the launch path reads the environment; the two
 * environment switches of a handle (KRAKEN_NO_GRAPH, KRAKEN_DECODE_ONE_CHAIN) are read once by kraken_create.
 * Errors: EINVAL (unknown key, value outside 0..3). */
typedef enum kraken_tuning_key {
    KRAKEN_TUNE_LN_ROW_KERNEL = 0,   /* LayerNorm of few or wide rows: 1 = one warp per row, 2 = one CTA per row */
    KRAKEN_TUNE_ATTN_SCHEDULE = 1,   /* prefill attention: 1 = one CTA per work item (no per-CTA work lists)     */
    KRAKEN_TUNE_LN_FUSION = 2,       /* LayerNorm inside the kernel that finishes its input rows (kraken_op_grouped_gemm_ln):
                                        2 = wherever it fits, 3 = behind the FFN down-projection only; 0, 1 = every
                                        LayerNorm its own launch (the default: see the measurements in the source)   */
    KRAKEN_TUNE_LAST_LAYER = 3,      /* prefill that returns last-position logits: 1 = the last layer runs on every row too */
    KRAKEN_TUNE_COUNT = 4
} kraken_tuning_key;
int kraken_tuning_set(int32_t key, int32_t value);

/* Makes one bounded wait run out, harmlessly: a single small CTA waits, with the library's own wait routine
 * and a limit of limit_us microseconds (1 .. 1,000,000), on a barrier that nothing ever signals and that has
 * no copy in flight, then takes the same way out as the model kernels do: it returns normally and raises
 * bit 1 of *d_status (device uint32).  Asynchronous on `stream`; the context stays usable.  This is how
 * the failure path of the kernels' waits (Sec. 3.1's steps never block forever here) is exercised
 * without starving a real kernel.  Errors: EINVAL, ECUDA. */
int kraken_test_wait_limit(uint32_t *d_status, uint32_t limit_us, void *stream);

/* Issue-rate probe for the tensor-core products of the attention step (Sec. 2.1's softmax(Q K^T) V on 128 x 128
 * tiles): n_ctas CTAs (one per SM at most) each issue `iters` blocks of `tcgen05.mma` instructions of M 128,
 * K 16 from one thread (issuers = 1) or from two threads in different warps (issuers = 2, each on its own
 * accumulator) and record the SM clock cycles from the first issue to the completion of the last product in
 * d_cycles[cta] (device int64; -1 if a bounded wait gave up, then bit 1 of *d_status is raised too).
 * form: 0 = S = Q K^T (both operands in shared memory, N 128); 1 = O += P V (A from tensor memory, V MN-major in
 * shared memory, N 128); 2 = 8 of the first then 8 of the second, alternating (the attention kernel's pattern);
 * 3 = form 2 with a commit after every 8; 4 = form 3 with a barrier wait that succeeds at once after every 8;
 * 5 = form 0 with N 64; 6 = form 0 with N 256.  *products_per_iter (host, may be NULL) receives the products one
 * thread issues per iteration, so cycles per product = d_cycles / (iters * products_per_iter) for one issuer and
 * half of that for two.  A measurement tool, not part of the model's arithmetic.  Errors: EINVAL, ECUDA. */
int kraken_test_mma_issue_rate(int32_t form, int32_t issuers, int32_t iters, int64_t *d_cycles, int32_t n_ctas,
                               int32_t *products_per_iter, uint32_t *d_status, void *stream);

/* ------------------------------------------------------------------------------------------
 * Single steps of the path, exposed so that each kernel can be checked on its own.  All
 * pointers are device pointers.  G is the number of groups (branches); a group stride of 0
 * shares one tensor between all groups.
 * ------------------------------------------------------------------------------------------ */

/* Shared embedding (Sec. 3.1): out[t, :] = wte[id[t], :] + wpe[pos0 + t % seqlen, :], fp32 [T, d].
 * d_status: device uint32, bit 0 is set when an id is outside [0, vocab) (that id reads row 0). */
int kraken_op_embed(const int32_t *d_ids, int32_t n_tokens, int32_t seqlen, int32_t pos0, const void *wte,
                    const void *wpe, int32_t d_model, int32_t vocab, float *d_out, uint32_t *d_status,
                    void *stream);

/* LayerNorm of Algorithm 1, both placements: out_g = LN(a_g + y; gamma_g, beta_g) -> bf16 [G][rows, d].
 * a: fp32 [G][rows, d] with group stride a_gstride elements (0 = shared); y: fp32 [rows, d] or NULL;
 * gamma/beta bf16 [G][d] (beta may be NULL).  d_status: device uint32 or NULL; with a status word
 * and many rows a persistent kernel with bounded waits is used (bit 1 = a wait ran out), without
 * one the warp-per-row kernel; both give the same bits. */
int kraken_op_layernorm(const float *d_a, int64_t a_gstride, const float *d_y, const void *gamma,
                        const void *beta, int32_t groups, int32_t rows, int32_t d_model, float eps,
                        void *d_out_bf16, uint32_t *d_status, void *stream);

/* Epilogues of the grouped GEMM  C_g = A_g . W_g^T (+ bias_g) ; A bf16 [G][M, K], W bf16 [G][Nout, K]. */
typedef enum kraken_epilogue {
    KRAKEN_EPI_F32 = 0,       /* out_f32[g] = acc + bias                                              */
    KRAKEN_EPI_BF16 = 1,      /* out_bf16[g] = bf16(acc + bias)                                       */
    KRAKEN_EPI_GELU_BF16 = 2, /* out_bf16[g] = bf16(GELU(acc + bias))             (FFN up-projection)  */
    KRAKEN_EPI_RESID_F32 = 3, /* out_f32[g] = resid[g] + acc + bias               (x = res + MHA(x))   */
    KRAKEN_EPI_RESID_SUM = 4, /* out_f32[g] = resid[g] + acc + bias; sum = SUM_g out_f32[g]
                                 (out = res + FFN(x), then the AllReduce of Algorithm 1)              */
    KRAKEN_EPI_QKV = 5        /* cols [0,d): out_bf16[g] (queries); [d,2d), [2d,3d): K, V rows written
                                 into the cache at [b][head][pos0 + t][dim], b = row / seqlen         */
} kraken_epilogue;

typedef struct kraken_gemm_args {
    const void *a;       int64_t a_gstride;    int32_t lda;   /* bf16 [G][M, K], row stride lda elements     */
    const void *w;       int64_t w_gstride;    int32_t ldw;   /* bf16 [G][Nout, K]                            */
    const void *bias;    int64_t bias_gstride;                /* bf16 [G][Nout] or NULL                       */
    int32_t groups, m, n_out, k;
    int32_t epilogue;                                         /* kraken_epilogue                              */
    float *out_f32;      int64_t out_f32_gstride;  int32_t ld_out_f32;
    void *out_bf16;      int64_t out_bf16_gstride; int32_t ld_out_bf16;
    const float *resid;  int64_t resid_gstride;    int32_t ld_resid; /* may alias out_f32 element for element  */
    float *sum;          int32_t ld_sum;                      /* fp32 [M, Nout], RESID_SUM only               */
    void *k_cache, *v_cache; int64_t cache_gstride;           /* QKV only: bases of this layer's K and V      */
    int32_t seqlen, pos0, n_head, head_dim, max_pos;          /* QKV only                                     */
    int32_t gelu_tanh;
    int32_t n_tile;                                           /* N tile: 0 = automatic; 32, 64, ... 256 (multiples of
                                                                 32) = one CTA per 128 x n_tile tile; 512 = CTA
                                                                 pairs on 256 x 256 tiles; 8 = the
                                                                 weight-streaming kernel for m <= 32 (no RESID_SUM) */
    int32_t n_kv_head;                                        /* QKV only: key/value heads (0 = n_head); the K and V
                                                                 parts of n_out are n_kv_head * head_dim wide each */
    int32_t w_constant;                                       /* nonzero: w holds constant data (weights), written by
                                                                 nothing queued on the stream before this call; the
                                                                 kernel then fetches its first W tiles while the
                                                                 stream's previous kernel is still finishing */
} kraken_gemm_args;

/* Grouped bf16 GEMM on the tensor cores (tcgen05 + TMEM accumulators, TMA operand loads).
 * Requirements: a, w 16-byte aligned; lda, ldw multiples of 8; k >= 8.  d_status as above (bit 1).
 * Errors: EINVAL, EUNSUPPORTED, ECUDA. */
int kraken_op_grouped_gemm(const kraken_gemm_args *args, uint32_t *d_status, void *stream);

/* LayerNorm of the finished rows in the same kernel as a RESID_F32 or RESID_SUM grouped GEMM (Algorithm 1:
 * `x = LN(x)` follows `out = res + FFN(x)`, `x = LN(x + y)` follows `x = res + MHA(x)`):
 *     ln_out[g] = LN(out_f32[g] + y; gamma[g], beta[g])      over the n_out columns of every row,
 * biased variance, statistics in fp32, result stored in the library's 16-bit type.  A row is spread over the
 * N tiles of its row block, i.e. over several CTAs: every epilogue warp leaves the statistics of its part in
 * d_scratch, waits (bounded; status bit 1 if it gives up) for the other parts and normalises the values it kept
 * in tensor memory.  out_f32 (and sum) are written as without the LayerNorm.
 * d_scratch: device memory of kraken_gemm_ln_scratch_bytes() bytes, zeroed ONCE by the caller before its first
 * use; every launch leaves its counters at zero again, so launches on one stream can share it (launches that
 * overlap on the device cannot; after a launch whose wait gave up, status bit 1, zero the scratch again).  gamma, beta: [G][n_out] (beta may be NULL = zeros); y: fp32 [M, n_out] added
 * to every group's rows before the statistics, or NULL.  Errors: EINVAL (other epilogues, missing pointers),
 * EUNSUPPORTED (m <= 32 rows with n_tile = 8; a row block of more N tiles than CTAs run at once),
 * ECAPACITY (scratch_bytes too small). */
typedef struct kraken_gemm_ln_args {
    void *ln_out;        int64_t ln_out_gstride; int32_t ld_ln_out;   /* 16-bit [G][M, n_out]                 */
    const void *gamma;   const void *beta;       int64_t gb_gstride;  /* 16-bit [G][n_out]                    */
    const float *y;      int32_t ld_y;
    float eps;
    void *d_scratch;     size_t scratch_bytes;
} kraken_gemm_ln_args;
int kraken_gemm_ln_scratch_bytes(int32_t groups, int32_t m, int32_t n_out, int32_t k, int32_t n_tile, size_t *bytes);
int kraken_op_grouped_gemm_ln(const kraken_gemm_args *args, const kraken_gemm_ln_args *ln, uint32_t *d_status,
                              void *stream);

/* Causal multi-head attention over a prefix held in the cache layout (Sec. 2.1):
 * for sequence b, head h, query row t (position pos0 + t): softmax over keys 0..pos0+t of
 * q.k / sqrt(head_dim), times V.  q, out: bf16 [G][batch*seqlen, n_head*head_dim];
 * k_cache, v_cache: bf16 [G][.][batch_stride][n_kv_head][max_pos][head_dim] as described by
 * cache_gstride / cache_bstride (elements).  n_kv_head: key/value heads in the cache, 0 = n_head;
 * with fewer (grouped-query / multi-query attention) query head h reads key/value head
 * h / (n_head / n_kv_head). */
int kraken_op_attention(const void *q, int64_t q_gstride, const void *k_cache, const void *v_cache,
                        int64_t cache_gstride, int64_t cache_bstride, int32_t groups, int32_t batch,
                        int32_t seqlen, int32_t pos0, int32_t n_head, int32_t n_kv_head, int32_t head_dim,
                        int32_t max_pos, void *out, int64_t out_gstride, void *stream);

/* Decode-step attention (Sec. 2.1: the decode step reads the whole KV cache): one query row per
 * (group, sequence, head) at position n_keys - 1 against cache rows 0..n_keys-1.  The keys are split
 * over `splits` CTAs per (group, sequence, head); each split leaves an unnormalised partial in
 * d_partials (device scratch, fp32 [groups*batch*n_head][splits][head_dim + 2]) and a second kernel
 * merges them.  splits = 0 lets the library choose; splits = 1 needs no scratch (d_partials may be NULL).
 * q, out: bf16 [G][batch, n_head*head_dim].  n_kv_head as in kraken_op_attention: the query heads of a
 * group are served together, so each cache row is fetched once per group.  Errors: EINVAL,
 * EUNSUPPORTED (head_dim), ECAPACITY (partial_bytes too small). */
int kraken_op_decode_attention(const void *q, int64_t q_gstride, const void *k_cache, const void *v_cache,
                               int64_t cache_gstride, int64_t cache_bstride, int32_t groups, int32_t batch,
                               int32_t n_keys, int32_t n_head, int32_t n_kv_head, int32_t head_dim, int32_t max_pos,
                               int32_t splits, void *d_partials, size_t partial_bytes, void *out,
                               int64_t out_gstride, void *stream);

/* Split count the library would choose (when *splits == 0 on entry; otherwise *splits is validated and kept)
 * and the scratch bytes kraken_op_decode_attention needs for it.  Pure host arithmetic. */
int kraken_decode_attention_sizes(int32_t groups, int32_t batch, int32_t n_keys, int32_t n_head, int32_t head_dim,
                                  int32_t *splits, size_t *partial_bytes);

/* (The paper has no counterpart to this call; it exists for hosts that cannot allocate.)
 * kraken_op_decode_attention without a scratch argument.  Meant for callers that have no way to
 * give the library device memory of their own: servers whose memory pool already owns the whole
 * device so that a fresh cudaMalloc fails, plugin-style integrations that are handed only input and
 * output pointers, and loops that cannot afford the device-wide synchronisation an allocation
 * implies.  The split-KV partials go to a fixed 8 MiB array inside the library image (held by every
 * GPU that loads the library, until the process exits); the call itself allocates nothing, on the
 * host side of CUDA or on the device.
 *   - Same layouts and results as kraken_op_decode_attention with n_kv_head = n_head (q, out: device bf16
 *     [G][batch, n_head*head_dim]; caches as there with one key/value head per query head: there is no
 *     grouped-query form of this call; splits = 0 lets the library choose); the same head dims are
 *     accepted (64, 72, 96, 104, 128; EUNSUPPORTED otherwise).
 *   - ECAPACITY when groups * batch * n_head * splits * (head_dim + 2) * 4 bytes exceeds
 *     kraken_decode_attention_static_capacity(); pass a smaller `splits` (1 needs no partials).
 *   - The first call on each device looks up the array's device address (once per device, with that
 *     device current); make that first call before starting any stream capture.  On EVERY call the
 *     current device must be the one that owns `stream`, q and out: the array is per device, and
 *     the call checks where q lives and returns EINVAL when that is another device.
 *   - All calls share the one array and it keeps whatever the previous call left.  Nothing in it has
 *     to start at zero: each call overwrites every partial it later reads.  Two calls whose kernels
 *     may overlap on the GPU (different streams) race on it; serialise them. */
int kraken_op_decode_attention_static(const void *q, int64_t q_gstride, const void *k_cache, const void *v_cache,
                                      int64_t cache_gstride, int64_t cache_bstride, int32_t groups, int32_t batch,
                                      int32_t n_keys, int32_t n_head, int32_t head_dim, int32_t max_pos,
                                      int32_t splits, void *out, int64_t out_gstride, void *stream);
size_t kraken_decode_attention_static_capacity(void);

#ifdef __cplusplus
}
#endif
#endif /* KRAKEN_H_ */
