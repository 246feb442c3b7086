// The C ABI: configuration checks, handle, and the kernel sequence of prefill / decode.
//
// kraken_prefill enqueues, on the caller's stream, with no host synchronisation:
//   embed -> for every layer { LN1[N] -> GEMM qkv[N] (K,V scattered into the cache) -> attention[N,B,H]
//            -> GEMM proj[N] (+bias +residual) -> LN2[N] on (a_n + y) -> GEMM up[N] (+bias, GELU)
//            -> GEMM down[N] (+bias +residual, cross-branch sum -> y of the next layer) }
//   -> gather of the wanted rows -> GEMM W_concat -> final LN -> GEMM unembedding -> fp32 logits.
#include <string.h>

#include <algorithm>

#include <new>
#include <vector>

#include "internal.h"
#include "ptx.cuh"

using namespace kr;

namespace {

constexpr size_t ALIGN = 256;
size_t align_up(size_t v) { return (v + ALIGN - 1) / ALIGN * ALIGN; }

struct Layout {
    size_t status, tokens, rows, logits, x0, x, a, s, u, q, o, g, dec_part, x_alt, row_seq, row_pos, pos_arr, ln_parts,
        ln_parts_bytes, ln_cnt, ln_cnt_bytes, last_q, last_o, last_a, last_x, last_y, last_u, last_g, last_r, last_len, total;
};

int kv_heads_of(const kraken_config &c) { return c.n_kv_head > 0 ? c.n_kv_head : c.n_head; }

int check_config(const kraken_config *c) {
    if (!c) return KRAKEN_EINVAL;
    if (c->n_branch < 1 || c->n_layer < 1 || c->d_model < 1 || c->n_head < 1 || c->d_ff < 1 || c->vocab < 1 ||
        c->max_pos < 1 || c->max_batch < 1 || !(c->ln_eps > 0.f))
        return KRAKEN_EINVAL;
    if (c->d_model % c->n_head != 0) return KRAKEN_EINVAL;
    if (c->n_kv_head < 0 || (c->n_kv_head > 0 && c->n_head % c->n_kv_head != 0)) return KRAKEN_EINVAL;
    if (c->parallel_ffn && !c->no_combine) return KRAKEN_EINVAL;   // the parallel variant has no cross-branch term
    const int hd = c->d_model / c->n_head;
    // 64 and 128, and the head dims of the paper's engine shapes (Table 3: 72, 96, 104)
    if (hd != 64 && hd != 72 && hd != 96 && hd != 104 && hd != 128) return KRAKEN_EUNSUPPORTED;
    // rows of every operand are multiples of 16 bytes (TMA strides, vector accesses)
    if (c->d_model % 8 != 0 || c->d_ff % 8 != 0) return KRAKEN_EUNSUPPORTED;
    return KRAKEN_OK;
}

size_t kv_bytes_of(const kraken_config *c) {
    return (size_t)c->n_layer * c->n_branch * 2 * c->max_batch * c->max_pos *
           (size_t)(kv_heads_of(*c) * (c->d_model / c->n_head)) * 2;
}

Layout layout_of(const kraken_config *c) {
    const size_t T = (size_t)c->max_batch * c->max_pos, d = c->d_model, N = c->n_branch, F = c->d_ff;
    Layout l;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off += align_up(bytes);
        return o;
    };
    l.status = take(256);
    l.tokens = take(T * 4);
    l.rows = take(T * 4);
    l.logits = take((size_t)c->max_batch * c->vocab * 4);
    l.x0 = take(T * d * 4);
    l.x = take(N * T * d * 4);
    l.a = take(N * T * d * 4);
    l.s = take(T * d * 4);
    l.u = take(N * T * d * 2);
    l.q = take(N * T * d * 2);
    l.o = take(N * T * d * 2);
    l.g = take(N * T * F * 2);
    l.dec_part = take(decode_attention_partial_bytes(c->n_branch, c->max_batch, c->n_head, c->d_model / c->n_head,
                                                     DECODE_MAX_SPLITS));
    l.x_alt = take((size_t)N * c->max_batch * d * 4);   // second copy of the branch outputs of a decode step
    l.row_seq = take(T * 4);                            // packed prefill: sequence and position of every row
    l.row_pos = take(T * 4);
    l.pos_arr = take((size_t)c->max_batch * 4);         // next position of every sequence (device copy)
    // LayerNorm behind the GEMM epilogues: per row and N tile two (mean, M2, count) entries, and two counters per
    // 32 rows.  Sized for 256-wide tiles on every row; narrower tiles (short prompts) fit into the 4 MiB floor or
    // the LayerNorm runs as its own launch.
    l.ln_parts_bytes = std::max<size_t>(gemm_ln_parts_bytes((int)N, (int)T, (int)d, GEMM_TILE_PAIR), size_t(4) << 20);
    l.ln_parts = take(l.ln_parts_bytes);
    l.ln_cnt_bytes = gemm_ln_cnt_bytes((int)N, (int)T);
    l.ln_cnt = take(l.ln_cnt_bytes);
    // the last layer of a prefill that only returns last-position logits: one row per sequence past the qkv GEMM
    const size_t Bm = c->max_batch;
    l.last_q = take(N * Bm * d * 2);
    l.last_o = take(N * Bm * d * 2);
    l.last_a = take(N * Bm * d * 4);
    l.last_x = take(N * Bm * d * 4);
    l.last_y = take(Bm * d * 4);
    l.last_u = take(N * Bm * d * 2);
    l.last_g = take(N * Bm * F * 2);
    l.last_r = take(N * Bm * d * 4);
    l.last_len = take(Bm * 4);
    l.total = off;
    return l;
}

enum GemmKind { G_QKV = 0, G_PROJ, G_UP, G_DOWN, G_CONCAT, G_HEAD, G_COUNT };

}  // namespace

constexpr int MAX_CHAINS = 8;

struct kraken_handle {
    kraken_config cfg;
    kraken_weights w;
    uint8_t *kv;
    uint8_t *scratch;
    Layout lay;
    int cur_len, batch, last_seqlen, last_rows;  // last_rows: token rows of the last model run
    // the last prefill ran its last layer, past the qkv GEMM, for the last position of every sequence only: the
    // layer outputs of the other rows are not there (kraken_logits_rows completes the layer first)
    bool x_partial;
    // length of every cached sequence (cur_len is their maximum); ragged = they differ, set by a packed prefill
    std::vector<int> seq_len;
    bool ragged;
    int stage_layer_done;   // branch-parallel driving: the last layer whose FFN half has run (-1: none)
    bool stage_decode;      // the pieces being driven are a decode step (one new token per sequence)
    std::vector<int> host_rows, host_row_seq, host_row_pos, host_len_m1;   // staging of the packed-prefill tables
    cudaStream_t last_stream;
    bool one_chain;   // decode steps keep all branches in one chain of launches (KRAKEN_DECODE_ONE_CHAIN at create)
    // weight tensor maps, one per GEMM kind, re-encoded when the N tile changes
    CUtensorMap tmB[G_COUNT];
    int tmB_bn[G_COUNT];
    // activation tensor maps, re-encoded when anything they describe changes (base, rows, groups, group stride)
    CUtensorMap tmA[G_COUNT];
    struct AKey { const void *base; int rows, groups; long long gstride; } tmA_key[G_COUNT];
    // decode steps replayed as a CUDA graph: positions are read from `pos` in device memory, tokens
    // and logits go through the staging buffers, so one graph serves every step of a batch size
    // a prefill with the same shape and buffers as the previous one is replayed as a graph too (it has a
    // fixed kernel sequence; worth it for short prompts, where launch gaps are a visible share)
    cudaGraphExec_t pre_graph;
    const void *pre_tokens, *pre_logits;
    int pre_batch, pre_seqlen, pre_all, pre_seen;
    long long pre_graph_launches[KRAKEN_PROF_COUNT];
    cudaGraphExec_t dec_graph;
    cudaStream_t cap_stream;                  // capture happens here (the caller's stream may be the legacy default)
    int dec_graph_batch;
    int dec_eager_steps;                      // eager steps done for the current batch size (warm-up)
    long long dec_graph_launches[KRAKEN_PROF_COUNT];
    bool use_graph;
    // decode steps run the branches as concurrent chains, one stream each (see run_layers_decode_branches)
    cudaStream_t br_stream[MAX_CHAINS];
    cudaEvent_t ev_fork, ev_join[MAX_CHAINS], ev_down[2][MAX_CHAINS];
    bool br_ready;
    // launch accounting and optional per-kernel timing
    long long launches[KRAKEN_PROF_COUNT];
    bool prof_on;
    std::vector<cudaEvent_t> ev_pool;
    size_t ev_used;
    struct Span { int cat; size_t e0, e1; };
    std::vector<Span> spans;
};

namespace {

template <typename T>
T *at(kraken_handle *h, size_t off) {
    return reinterpret_cast<T *>(h->scratch + off);
}

cudaEvent_t prof_event(kraken_handle *h) {
    if (h->ev_used == h->ev_pool.size()) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
        h->ev_pool.push_back(e);
    }
    return h->ev_pool[h->ev_used++];
}

// Counts a kernel launch of category `cat`; with profiling on, brackets it with events.
struct LaunchScope {
    kraken_handle *h;
    cudaStream_t st;
    bool timed;
    LaunchScope(kraken_handle *h_, int cat, cudaStream_t st_) : h(h_), st(st_), timed(false) {
        h->launches[cat]++;
        if (h->prof_on) {
            cudaEvent_t e0 = prof_event(h), e1 = prof_event(h);
            if (e0 && e1) {
                cudaEventRecord(e0, st);
                h->spans.push_back({cat, h->ev_used - 2, h->ev_used - 1});
                timed = true;
            }
        }
    }
    ~LaunchScope() {
        if (timed) cudaEventRecord(h->ev_pool[h->spans.back().e1], st);
    }
};

struct RunCtx {
    kraken_handle *h;
    cudaStream_t st;
    int batch, seqlen, pos0, T;
    const int *pos_dev;  // decode: the next position of every sequence, in device memory
    int max_keys;        // decode: upper bound of the keys a step can see (fixes the split count)
    // packed prefill of sequences of different lengths (h->seq_len): sequence and position of every row;
    // seqlen is then the longest length
    bool packed;
    const int *row_seq, *row_pos;
    // branch-parallel deployment: the path is driven in pieces (kraken_stage_*): 0 = the whole path,
    // STAGE_EMBED, STAGE_ATTN / STAGE_FFN = one half of layer stage_layer; y_ext = the cross-device sum for LN2
    int stage, stage_layer;
    const float *y_ext;
    // TTFT needs the logits of the last position of every sequence only, so the last layer's attention queries and
    // everything after them (output projection, LN-2, FFN) are needed for those rows only; K and V of the last layer
    // are still computed for every position (the cache).  last_rows: device list of those rows, one per sequence.
    bool last_only = false;
    const int32_t *last_rows = nullptr;
    const int *last_len_m1 = nullptr;   // packed prefill: length - 1 of every sequence (device), else all are seqlen - 1
    int only_layer = -1;   // >= 0: run this layer alone, on every row (completing a last_only prefill)
};
enum { STAGE_ALL = 0, STAGE_EMBED = 1, STAGE_ATTN = 2, STAGE_FFN = 3 };

// One grouped GEMM of the model: weights of `kind` at `layer`.
// g0 / gcnt: a run of branches (gcnt = 0: all of them; the caller then passes A and the epilogue's pointers
// already moved to branch g0); st: the stream (null: the call's stream).
int model_gemm(const RunCtx &rc, GemmKind kind, int layer, int m_rows, const uint16_t *a, long long a_gstride,
               EpiParams epi, int g0 = 0, int gcnt = 0, cudaStream_t st = nullptr) {
    kraken_handle *h = rc.h;
    const kraken_config &c = h->cfg;
    const int d = c.d_model, F = c.d_ff, N = c.n_branch;
    GemmOperands op;
    GemmShape s;
    int total_groups;  // groups held by the weight tensor across all layers
    const uint16_t *wbase;
    const uint16_t *bias = nullptr;
    switch (kind) {
        case G_QKV: s = {N, m_rows, d + 2 * kv_heads_of(c) * (d / c.n_head), d}; wbase = (const uint16_t *)h->w.w_qkv; bias = (const uint16_t *)h->w.b_qkv; break;
        case G_PROJ: s = {N, m_rows, d, d}; wbase = (const uint16_t *)h->w.w_proj; bias = (const uint16_t *)h->w.b_proj; break;
        case G_UP: s = {N, m_rows, F, d}; wbase = (const uint16_t *)h->w.w_up; bias = (const uint16_t *)h->w.b_up; break;
        case G_DOWN: s = {N, m_rows, d, F}; wbase = (const uint16_t *)h->w.w_down; bias = (const uint16_t *)h->w.b_down; break;
        case G_CONCAT: s = {1, m_rows, d, N * d}; wbase = (const uint16_t *)h->w.w_concat; bias = (const uint16_t *)h->w.b_concat; break;
        default: s = {1, m_rows, c.vocab, d}; wbase = (const uint16_t *)h->w.wte; break;
    }
    const bool layered = kind <= G_DOWN;
    total_groups = layered ? c.n_layer * N : 1;
    if (gcnt > 0) s.groups = gcnt;
    if (!st) st = rc.st;
    const long long w_gstride = (long long)s.n_out * s.k;
    op.a = a;
    op.a_gstride = a_gstride;
    op.lda = s.k;
    op.ldw = s.k;
    op.w_gstride = w_gstride;
    op.w = wbase + (layered ? ((long long)layer * N + g0) * w_gstride : 0);
#ifndef KR_W_EARLY
#define KR_W_EARLY 1
#endif
    op.w_static = KR_W_EARLY != 0;
    if (bias) {
        epi.bias = bias + (layered ? ((long long)layer * N + g0) * s.n_out : 0);
        epi.bias_gstride = s.n_out;
    } else {
        epi.bias = nullptr;
        epi.bias_gstride = 0;
    }
    static const int cat_of[G_COUNT] = {KRAKEN_PROF_GEMM_QKV, KRAKEN_PROF_GEMM_PROJ, KRAKEN_PROF_GEMM_UP,
                                        KRAKEN_PROF_GEMM_DOWN, KRAKEN_PROF_TAIL, KRAKEN_PROF_TAIL};
    LaunchScope scope(h, cat_of[kind], st);
    if (m_rows <= SKINNY_MAX_ROWS && epi.kind != KRAKEN_EPI_RESID_SUM) return launch_gemm_skinny(op, s, epi, st);

    const int bn = gemm_pick_bn(s);
    if (h->tmB_bn[kind] != bn) {
        GemmOperands all = op;
        all.w = wbase;
        GemmShape sa = s;
        sa.groups = total_groups;
        int r = gemm_encode_b(&h->tmB[kind], all, sa, bn);
        if (r) return r;
        h->tmB_bn[kind] = bn;
    }
    // A maps: the up-projection reads the same buffer as qkv but after LN2, same shape -> same map works.
    // (a run of branches starting at g0 > 0 has its own base pointer, so it never reuses another run's map)
    const kraken_handle::AKey key{a, m_rows, s.groups, a_gstride};
    kraken_handle::AKey &have = h->tmA_key[kind];
    if (have.base != key.base || have.rows != key.rows || have.groups != key.groups || have.gstride != key.gstride) {
        int r = gemm_encode_a(&h->tmA[kind], op, s);
        if (r) return r;
        have = key;
    }
    return launch_gemm_tc(op, s, epi, &h->tmA[kind], &h->tmB[kind], layered ? layer * N + g0 : 0, bn,
                          at<uint32_t>(h, h->lay.status), st);
}

EpiParams epi_zero() {
    EpiParams e;
    memset(&e, 0, sizeof(e));
    return e;
}

#define KR_TRY(x)            \
    do {                     \
        int _rc = (x);       \
        if (_rc) return _rc; \
    } while (0)

int branch_streams(kraken_handle *h);

#define KR_CU(x)                                              \
    do {                                                      \
        if ((x) != cudaSuccess) return cuda_check(cudaGetLastError(), "streams and events"); \
    } while (0)

// Whether this run takes the short form of the last layer (see RunCtx::last_only): a whole-path prefill with more
// than 32 rows (shorter prompts do not form the cross-branch sum as a tensor).
bool short_last_of(const RunCtx &rc) {
    return rc.last_only && !rc.stage && rc.only_layer < 0 && rc.T > SKINNY_MAX_ROWS && rc.last_rows != nullptr &&
           (!rc.packed || rc.last_len_m1 != nullptr);
}

// Runs the L layers on `T = batch * seqlen` new tokens at positions pos0 .. pos0 + seqlen - 1.
int run_layers(const RunCtx &rc, const int32_t *d_tokens) {
    kraken_handle *h = rc.h;
    const kraken_config &c = h->cfg;
    const int d = c.d_model, F = c.d_ff, N = c.n_branch, L = c.n_layer, H = c.n_head, hd = d / H, T = rc.T;
    const long long td = (long long)T * d;
    // The down-projection's epilogue can form the cross-branch sum only by running the N groups of an
    // output tile on one CTA (pair); with too few output tiles that would idle most SMs, so then (and in
    // decode) LayerNorm-2 of the next layer sums the N branch inputs itself, in the same order.
    const long long down_tiles = (long long)((T + 255) / 256) * ((d + 255) / 256);
    const bool small_rows = (T <= SKINNY_MAX_ROWS || down_tiles < (sm_count() > 0 ? sm_count() : 148) / 2);
    // between the two: all groups of the down-projection run side by side and one streaming pass adds the N outputs
    const bool sum_pass = small_rows && T > SKINNY_MAX_ROWS;
    const bool sum_beside = sum_pass && !rc.stage && branch_streams(h) == KRAKEN_OK;
    bool sum_pending = false;
    uint16_t *const u_ = at<uint16_t>(h, h->lay.u);
    // A LayerNorm can run behind the epilogue of the GEMM that finishes its input rows (LN-2 behind the attention
    // output projection, the next layer's LN-1 behind the down-projection) when that GEMM goes to the tensor-core
    // kernels, the statistics scratch holds its tiling and the path is not driven in pieces (there y comes from
    // outside after the projection).  It is not the default: measured, it pays only behind the down-projection of
    // long prompts (K = d_ff per tile leaves the epilogue time to spare: C3 109.4 -> 108.9 ms), costs time behind
    // the output projection (its epilogue already bounds it: 8.2 -> 18.6 ms per step) and for short prompts (one
    // tile per CTA, the wait for the row block's other tiles is exposed: C1 0.98 -> 1.04 ms), and the statistics
    // are summed in another order than the LayerNorm kernel's, so a sequence would no longer give the same 16-bit
    // activations alone and inside a batch that takes the other route.  KRAKEN_TUNE_LN_FUSION: 2 = wherever it
    // fits, 3 = behind the down-projection only.  The first layer's LN-1 reads the embedding and is always a
    // launch of its own.
    auto ln_fits = [&](const GemmShape &gs) {
        const int bn = gemm_pick_bn(gs);
        const int cols = bn == GEMM_TILE_PAIR ? 256 : bn;
        const int sms = sm_count() > 0 ? sm_count() : 148;
        return gemm_ln_parts_bytes(N, T, d, bn) <= h->lay.ln_parts_bytes &&
               (d + cols - 1) / cols <= (bn == GEMM_TILE_PAIR ? sms / 2 : sms);
    };
    const int ln_mode = tuning(KRAKEN_TUNE_LN_FUSION);
    const bool ln_fuse = !rc.stage && T > SKINNY_MAX_ROWS && (ln_mode == 2 || ln_mode == 3);
    const bool fuse_ln2 = ln_fuse && ln_mode == 2 && !c.parallel_ffn && ln_fits(GemmShape{N, T, d, d});
    const bool fuse_ln1 = ln_fuse && ln_fits(GemmShape{N, T, d, F});
    auto ln_epi = [&](EpiParams &e, const void *gamma, const void *beta, long long off, const float *y) {
        e.ln_out = u_; e.ln_out_gstride = td; e.ln_ld_out = d;
        e.ln_gamma = (const uint16_t *)gamma + off;
        e.ln_beta = beta ? (const uint16_t *)beta + off : nullptr;
        e.ln_gb_gstride = d;
        e.ln_y = y; e.ln_ld_y = d;
        e.ln_eps = c.ln_eps;
        e.ln_parts = at<float4>(h, h->lay.ln_parts);
        e.ln_cnt = at<uint32_t>(h, h->lay.ln_cnt);
    };
    float *x0 = at<float>(h, h->lay.x0), *x = at<float>(h, h->lay.x), *a = at<float>(h, h->lay.a),
          *S = at<float>(h, h->lay.s);
    uint16_t *u = at<uint16_t>(h, h->lay.u), *q = at<uint16_t>(h, h->lay.q), *o = at<uint16_t>(h, h->lay.o),
             *gb = at<uint16_t>(h, h->lay.g);
    uint32_t *status = at<uint32_t>(h, h->lay.status);
    const int Hkv = kv_heads_of(c);
    const long long cache_b = (long long)Hkv * c.max_pos * hd;    // one sequence of one of K / V
    const long long cache_kv = (long long)c.max_batch * cache_b;  // all of K (or V) of one (layer, branch)
    uint16_t *kv = reinterpret_cast<uint16_t *>(h->kv);

    if ((rc.stage == STAGE_ALL && rc.only_layer < 0) || rc.stage == STAGE_EMBED) {
        LaunchScope scope(h, KRAKEN_PROF_EMBED, rc.st);
        KR_TRY(launch_embed(d_tokens, T, rc.seqlen, rc.pos0, (const uint16_t *)h->w.wte, (const uint16_t *)h->w.wpe, d,
                            c.vocab, x0, status, rc.st, rc.pos_dev, rc.row_pos));
    }
    if (rc.stage == STAGE_EMBED) return KRAKEN_OK;
    const int l_begin = rc.stage ? rc.stage_layer : (rc.only_layer >= 0 ? rc.only_layer : 0);
    const int l_end = rc.stage ? rc.stage_layer + 1 : (rc.only_layer >= 0 ? rc.only_layer + 1 : L);
    // (the short last layer needs the cross-branch sum as a tensor, which prompts of up to 32 rows do not form)
    const bool short_last = short_last_of(rc);
    for (int l = l_begin; l < l_end; ++l) {
        const float *xin = l == 0 ? x0 : x;
        const long long xin_gs = l == 0 ? 0 : td;
        const long long ln_off = (long long)l * N * d;
        EpiParams e = epi_zero();
        if (rc.stage != STAGE_FFN) {
        // x = LN(x)   (already done behind the previous layer's down-projection when fused)
        if (!(fuse_ln1 && l > l_begin)) {
            LaunchScope scope(h, KRAKEN_PROF_LAYERNORM, rc.st);
            KR_TRY(launch_layernorm(xin, xin_gs, nullptr, (const uint16_t *)h->w.ln1_g + ln_off,
                                    h->w.ln1_b ? (const uint16_t *)h->w.ln1_b + ln_off : nullptr, N, T, d, c.ln_eps,
                                    u, rc.st, nullptr, 0, 0, status));
        }
        // q | k | v ; K and V go straight into the cache
        uint16_t *kc = kv + (long long)l * N * 2 * cache_kv;
        e = epi_zero();
        e.kind = KRAKEN_EPI_QKV;
        e.out_bf16 = q; e.out_bf16_gstride = td; e.ld_out_bf16 = d;
        e.k_cache = kc; e.v_cache = kc + cache_kv; e.cache_gstride = 2 * cache_kv;
        e.seqlen = rc.seqlen; e.pos0 = rc.pos0; e.n_head = H; e.head_dim = hd; e.max_pos = c.max_pos; e.d_model = d;
        e.n_kv_head = Hkv;
        e.pos0_dev = rc.pos_dev;
        e.row_seq = rc.row_seq; e.row_pos = rc.row_pos;
        KR_TRY(model_gemm(rc, G_QKV, l, T, u, td, e));
        if (short_last && l == L - 1) {
            // Last layer, last position of every sequence only (K and V of every position are in the cache by now):
            // the rows' queries are gathered, attend over the cache like a decode step, and the rest of the layer
            // runs on batch rows.
            const int n = rc.batch;
            const long long nd = (long long)n * d;
            uint16_t *ql = at<uint16_t>(h, h->lay.last_q), *ol = at<uint16_t>(h, h->lay.last_o),
                     *ul = at<uint16_t>(h, h->lay.last_u), *gl = at<uint16_t>(h, h->lay.last_g);
            float *al = at<float>(h, h->lay.last_a), *xl = at<float>(h, h->lay.last_x), *yl = at<float>(h, h->lay.last_y),
                  *rl = at<float>(h, h->lay.last_r);
            {
                LaunchScope scope(h, KRAKEN_PROF_ATTENTION, rc.st);
                KR_TRY(launch_gather_rows(q, td * 2, N, d * 2, rc.last_rows, n, ql, rc.st));
            }
            {
                LaunchScope scope(h, KRAKEN_PROF_ATTENTION, rc.st);
                DecodeAttnParams dp;
                dp.q = ql; dp.q_gstride = nd;
                dp.k_cache = kc; dp.v_cache = kc + cache_kv;
                dp.cache_gstride = 2 * cache_kv; dp.cache_bstride = cache_b;
                dp.groups = N; dp.batch = n; dp.n_keys = rc.pos0 + rc.seqlen; dp.n_head = H; dp.head_dim = hd;
                dp.n_kv_head = Hkv;
                dp.max_pos = c.max_pos;
                dp.pos_dev = rc.packed ? rc.last_len_m1 : nullptr;   // sequences of different lengths: their own key counts
                dp.splits = decode_attention_splits(N, n, (hd == 64 || hd == 128) && decode_gqa_tile(H, Hkv) ? Hkv : H,
                                                    dp.n_keys);
                dp.partials = at<float>(h, h->lay.dec_part);
                dp.out = ol; dp.out_gstride = nd;
                h->launches[KRAKEN_PROF_ATTENTION] += dp.splits > 1 ? 1 : 0;
                KR_TRY(launch_attention_decode(dp, rc.st));
            }
            e = epi_zero();
            e.kind = KRAKEN_EPI_RESID_F32;
            e.out_f32 = al; e.out_f32_gstride = nd; e.ld_out_f32 = d;
            {
                LaunchScope scope(h, KRAKEN_PROF_GEMM_PROJ, rc.st);   // the residual rows of the output projection
                KR_TRY(launch_gather_rows(xin, xin_gs * 4, xin_gs ? N : 1, d * 4, rc.last_rows, n, rl, rc.st));
            }
            e.resid = rl; e.resid_gstride = xin_gs ? nd : 0; e.ld_resid = d;
            KR_TRY(model_gemm(rc, G_PROJ, l, n, ol, nd, e));
            if (c.parallel_ffn) {
                LaunchScope scope(h, KRAKEN_PROF_LAYERNORM, rc.st);
                KR_TRY(launch_gather_rows(u, td * 2, N, d * 2, rc.last_rows, n, ul, rc.st));
            } else {
                if (sum_pending) {
                    KR_CU(cudaStreamWaitEvent(rc.st, h->ev_join[1], 0));
                    sum_pending = false;
                }
                const float *ysrc = c.no_combine ? nullptr : (l == 0 ? x0 : S);
                if (ysrc) {
                    LaunchScope scope(h, KRAKEN_PROF_LAYERNORM, rc.st);
                    KR_TRY(launch_gather_rows(ysrc, 0, 1, d * 4, rc.last_rows, n, yl, rc.st));
                }
                LaunchScope scope(h, KRAKEN_PROF_LAYERNORM, rc.st);
                KR_TRY(launch_layernorm(al, nd, ysrc ? yl : nullptr, (const uint16_t *)h->w.ln2_g + ln_off,
                                        h->w.ln2_b ? (const uint16_t *)h->w.ln2_b + ln_off : nullptr, N, n, d, c.ln_eps,
                                        ul, rc.st, nullptr, 0, 0, status));
            }
            e = epi_zero();
            e.kind = KRAKEN_EPI_GELU_BF16;
            e.out_bf16 = gl; e.out_bf16_gstride = (long long)n * F; e.ld_out_bf16 = F; e.gelu_tanh = c.gelu_tanh;
            KR_TRY(model_gemm(rc, G_UP, l, n, ul, nd, e));
            e = epi_zero();
            e.kind = KRAKEN_EPI_RESID_F32;
            e.out_f32 = xl; e.out_f32_gstride = nd; e.ld_out_f32 = d;
            e.resid = al; e.resid_gstride = nd; e.ld_resid = d;
            KR_TRY(model_gemm(rc, G_DOWN, l, n, gl, (long long)n * F, e));
            continue;
        }
        // attention over the cached prefix
        AttnParams ap;
        ap.q = q; ap.q_gstride = td;
        ap.k_cache = kc; ap.v_cache = kc + cache_kv; ap.cache_gstride = 2 * cache_kv; ap.cache_bstride = cache_b;
        ap.groups = N; ap.batch = rc.batch; ap.seqlen = rc.seqlen; ap.pos0 = rc.pos0; ap.n_head = H; ap.head_dim = hd;
        ap.n_kv_head = Hkv;
        ap.max_pos = c.max_pos; ap.out = o; ap.out_gstride = td;
        {
            LaunchScope scope(h, KRAKEN_PROF_ATTENTION, rc.st);
            if (rc.packed) {
                // sequences of different lengths: one launch per sequence on its rows of the packed tensors
                long long row0 = 0;
                for (int b = 0; b < rc.batch; ++b) {
                    AttnParams sp = ap;
                    sp.batch = 1;
                    sp.seqlen = h->seq_len[b];
                    sp.q = q + row0 * d;
                    sp.out = o + row0 * d;
                    sp.k_cache = ap.k_cache + b * cache_b;
                    sp.v_cache = ap.v_cache + b * cache_b;
                    if (b > 0) h->launches[KRAKEN_PROF_ATTENTION]++;
                    KR_TRY(launch_attention_tc(sp, nullptr, nullptr, nullptr, status, rc.st));
                    row0 += h->seq_len[b];
                }
            } else if (rc.seqlen == 1) {
                // decode step: stream the cache with the split-KV kernel
                DecodeAttnParams dp;
                dp.q = q; dp.q_gstride = td;
                dp.k_cache = ap.k_cache; dp.v_cache = ap.v_cache;
                dp.cache_gstride = ap.cache_gstride; dp.cache_bstride = ap.cache_bstride;
                dp.groups = N; dp.batch = rc.batch; dp.n_keys = rc.pos0 + 1; dp.n_head = H; dp.head_dim = hd;
                dp.n_kv_head = Hkv;
                dp.max_pos = c.max_pos;
                dp.pos_dev = rc.pos_dev;
                dp.splits = decode_attention_splits(N, rc.batch, (hd == 64 || hd == 128) && decode_gqa_tile(H, Hkv) ? Hkv : H,
                                                    rc.pos_dev ? rc.max_keys : dp.n_keys);
                dp.partials = at<float>(h, h->lay.dec_part);
                dp.out = o; dp.out_gstride = td;
                h->launches[KRAKEN_PROF_ATTENTION] += dp.splits > 1 ? 1 : 0;
                KR_TRY(launch_attention_decode(dp, rc.st));
            } else {
                KR_TRY(launch_attention_tc(ap, nullptr, nullptr, nullptr, status, rc.st));
            }
        }
        // x = res + MHA(x)
        e = epi_zero();
        e.kind = KRAKEN_EPI_RESID_F32;
        e.out_f32 = a; e.out_f32_gstride = td; e.ld_out_f32 = d;
        e.resid = xin; e.resid_gstride = xin_gs; e.ld_resid = d;
        if (fuse_ln2) {
            // x = LN(x + y) behind this epilogue: y is the shared embedding in the first layer, the cross-branch sum
            // afterwards (formed by the previous down-projection, or by the pass beside it, joined here)
            if (sum_pending) {
                KR_CU(cudaStreamWaitEvent(rc.st, h->ev_join[1], 0));
                sum_pending = false;
            }
            ln_epi(e, h->w.ln2_g, h->w.ln2_b, ln_off, c.no_combine ? nullptr : (l == 0 ? x0 : S));
        }
        KR_TRY(model_gemm(rc, G_PROJ, l, T, o, td, e));
        }  // attention half
        if (rc.stage == STAGE_ATTN) continue;
        // x = LN(x + y): y is the shared embedding in the first layer, the cross-branch sum afterwards
        // (the parallel variant feeds the FFN with the first LayerNorm's output, still in u)
        if (rc.stage == STAGE_FFN) {
            // driven from outside: y is whatever the caller summed over all devices (layer 1: the embedding)
            LaunchScope scope(h, KRAKEN_PROF_LAYERNORM, rc.st);
            KR_TRY(launch_layernorm(a, td, rc.y_ext, (const uint16_t *)h->w.ln2_g + ln_off,
                                    h->w.ln2_b ? (const uint16_t *)h->w.ln2_b + ln_off : nullptr, N, T, d, c.ln_eps,
                                    u, rc.st, nullptr, 0, 0, status));
        } else if (!c.parallel_ffn && !fuse_ln2) {
            if (sum_pending) {
                KR_CU(cudaStreamWaitEvent(rc.st, h->ev_join[1], 0));
                sum_pending = false;
            }
            LaunchScope scope(h, KRAKEN_PROF_LAYERNORM, rc.st);
            // with few rows the cross-branch sum is formed here from the N branch inputs (same order as
            // the down-projection epilogue forms it for long prompts)
            const bool sum_here = small_rows && !sum_pass && l > 0 && !c.no_combine;
            KR_TRY(launch_layernorm(a, td, (sum_here || c.no_combine) ? nullptr : (l == 0 ? x0 : S),
                                    (const uint16_t *)h->w.ln2_g + ln_off,
                                    h->w.ln2_b ? (const uint16_t *)h->w.ln2_b + ln_off : nullptr, N, T, d, c.ln_eps,
                                    u, rc.st, sum_here ? x : nullptr, td, N, status));
        }
        // FFN up + GELU
        e = epi_zero();
        e.kind = KRAKEN_EPI_GELU_BF16;
        e.out_bf16 = gb; e.out_bf16_gstride = (long long)T * F; e.ld_out_bf16 = F; e.gelu_tanh = c.gelu_tanh;
        KR_TRY(model_gemm(rc, G_UP, l, T, u, td, e));
        // out = res + FFN ; the sum over branches (the AllReduce feeding the next layer) in the epilogue
        e = epi_zero();
        e.kind = (l + 1 < L && !small_rows && !c.no_combine && !rc.stage) ? KRAKEN_EPI_RESID_SUM : KRAKEN_EPI_RESID_F32;
        e.out_f32 = x; e.out_f32_gstride = td; e.ld_out_f32 = d;
        e.resid = a; e.resid_gstride = td; e.ld_resid = d;
        e.sum = S; e.ld_sum = d;
        if (fuse_ln1 && l + 1 < l_end)   // the next layer's x = LN(x) behind this epilogue
            ln_epi(e, h->w.ln1_g, h->w.ln1_b, ln_off + (long long)N * d, nullptr);
        KR_TRY(model_gemm(rc, G_DOWN, l, T, gb, (long long)T * F, e));
        if (rc.stage == STAGE_FFN) {
            // driven from outside: the sum of this device's branches, for the caller's all-reduce
            LaunchScope scope(h, KRAKEN_PROF_LAYERNORM, rc.st);
            KR_TRY(launch_sum_groups(x, td, N, td, S, rc.st));
        } else if (sum_pass && l + 1 < L && !c.no_combine) {
            // The sum is first read by the next layer's second LayerNorm, so it runs beside that layer's
            // attention half on a stream of its own (x is not written again, nor S read, before the join).
            if (sum_beside) {
                KR_CU(cudaEventRecord(h->ev_fork, rc.st));
                KR_CU(cudaStreamWaitEvent(h->br_stream[1], h->ev_fork, 0));
            }
            cudaStream_t ss = sum_beside ? h->br_stream[1] : rc.st;
            {
                LaunchScope scope(h, KRAKEN_PROF_LAYERNORM, ss);
                KR_TRY(launch_sum_groups(x, td, N, td, S, ss));
            }
            if (sum_beside) {
                KR_CU(cudaEventRecord(h->ev_join[1], ss));
                sum_pending = true;
            }
        }
    }
    h->last_rows = T;
    return KRAKEN_OK;
}

// Streams and events of the branch chains, created on first use.
int branch_streams(kraken_handle *h) {
    if (h->br_ready) return KRAKEN_OK;
    for (int b = 0; b < MAX_CHAINS; ++b) {
        if (cudaStreamCreateWithFlags(&h->br_stream[b], cudaStreamNonBlocking) != cudaSuccess) return KRAKEN_ECUDA;
        if (cudaEventCreateWithFlags(&h->ev_join[b], cudaEventDisableTiming) != cudaSuccess) return KRAKEN_ECUDA;
        for (int p = 0; p < 2; ++p)
            if (cudaEventCreateWithFlags(&h->ev_down[p][b], cudaEventDisableTiming) != cudaSuccess) return KRAKEN_ECUDA;
    }
    if (cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) != cudaSuccess) return KRAKEN_ECUDA;
    h->br_ready = true;
    return KRAKEN_OK;
}

// The layers of one decode step (one new token per sequence) with every branch as its own chain of
// launches on its own stream.  A decode layer alternates a bandwidth-bound kernel (attention streaming the
// KV cache) with a run of short latency-bound ones (LayerNorms, weight-streaming GEMMs of a few MB);
// launched for all branches at once the two kinds take turns and HBM idles during the second.  The
// branches of a Kraken layer depend on each other only through the cross-branch sum that LayerNorm-2
// reads (Algorithm 1), so here branch b's chain  LN1 -> qkv -> attention -> proj  runs ahead on its own
// and only its LN2 waits for the other branches' previous-layer outputs; the chains drift apart by
// themselves, so one branch's cache streaming overlaps the others' short kernels (starting them a kernel
// or more apart on purpose measured the same or worse).
// Branch outputs alternate between two buffers by layer: a chain that runs ahead writes layer l while
// another chain's LN2 still sums the outputs of layer l-1.
int run_layers_decode_branches(const RunCtx &rc, const int32_t *d_tokens) {
    kraken_handle *h = rc.h;
    const kraken_config &c = h->cfg;
    const int d = c.d_model, F = c.d_ff, N = c.n_branch, L = c.n_layer, H = c.n_head, hd = d / H, T = rc.T;
    const long long td = (long long)T * d;
    KR_TRY(branch_streams(h));
    float *x0 = at<float>(h, h->lay.x0), *a = at<float>(h, h->lay.a);
    float *xbuf[2] = {at<float>(h, h->lay.x), at<float>(h, h->lay.x_alt)};
    uint16_t *u = at<uint16_t>(h, h->lay.u), *q = at<uint16_t>(h, h->lay.q), *o = at<uint16_t>(h, h->lay.o),
             *gb = at<uint16_t>(h, h->lay.g);
    uint32_t *status = at<uint32_t>(h, h->lay.status);
    const int Hkv = kv_heads_of(c);
    const long long cache_b = (long long)Hkv * c.max_pos * hd;
    const long long cache_kv = (long long)c.max_batch * cache_b;
    uint16_t *kv = reinterpret_cast<uint16_t *>(h->kv);
    auto stream_of = [&](int b) { return b == 0 ? rc.st : h->br_stream[b]; };
    auto out_of = [&](int l) { return xbuf[(L - 1 - l) & 1]; };   // the last layer lands in the main buffer

    {
        LaunchScope scope(h, KRAKEN_PROF_EMBED, rc.st);
        KR_TRY(launch_embed(d_tokens, T, rc.seqlen, rc.pos0, (const uint16_t *)h->w.wte, (const uint16_t *)h->w.wpe, d,
                            c.vocab, x0, status, rc.st, rc.pos_dev, rc.row_pos));
    }
    KR_CU(cudaEventRecord(h->ev_fork, rc.st));
    for (int b = 1; b < N; ++b) KR_CU(cudaStreamWaitEvent(h->br_stream[b], h->ev_fork, 0));

    const int tile = (hd == 64 || hd == 128) && decode_gqa_tile(H, Hkv);
    // splits per (sequence, head) of one branch: about six CTAs per SM per branch launch, rounded to nearest
    // (measured at 16 x 16 streams of 2100 keys: 3 splits 2.98 ms per step, 2: 3.11, 4: 3.16, 1: 3.36)
    int splits;
    {
        const long long streams = (long long)rc.batch * (tile ? Hkv : H);
        const int n_keys = rc.pos_dev ? rc.max_keys : rc.pos0 + 1;
        const long long want = 6LL * (sm_count() > 0 ? sm_count() : 148);
        long long sp = (want + streams / 2) / streams;
        const long long by_len = (n_keys + 127) / 128;
        if (sp > by_len) sp = by_len;
        if (sp > DECODE_MAX_SPLITS) sp = DECODE_MAX_SPLITS;
        if (sp < 1) sp = 1;
        splits = static_cast<int>(sp);
    }
    const long long part_b = (long long)rc.batch * H * splits * (hd + 2);   // floats of partials per branch

    for (int l = 0; l < L; ++l) {
        const long long ln_off = (long long)l * N * d;
        float *xout = out_of(l);
        const float *xprev = l == 0 ? nullptr : out_of(l - 1);
        uint16_t *kc = kv + (long long)l * N * 2 * cache_kv;
        for (int b = 0; b < N; ++b) {
            cudaStream_t st = stream_of(b);
            const float *xin = l == 0 ? x0 : xprev + b * td;
            {
                LaunchScope scope(h, KRAKEN_PROF_LAYERNORM, st);
                KR_TRY(launch_layernorm(xin, 0, nullptr, (const uint16_t *)h->w.ln1_g + ln_off + (long long)b * d,
                                        h->w.ln1_b ? (const uint16_t *)h->w.ln1_b + ln_off + (long long)b * d : nullptr,
                                        1, T, d, c.ln_eps, u + b * td, st));
            }
            EpiParams e = epi_zero();
            e.kind = KRAKEN_EPI_QKV;
            e.out_bf16 = q + b * td; e.out_bf16_gstride = td; e.ld_out_bf16 = d;
            e.k_cache = kc + (long long)b * 2 * cache_kv; e.v_cache = e.k_cache + cache_kv; e.cache_gstride = 2 * cache_kv;
            e.seqlen = rc.seqlen; e.pos0 = rc.pos0; e.n_head = H; e.head_dim = hd; e.max_pos = c.max_pos; e.d_model = d;
            e.n_kv_head = Hkv;
            e.pos0_dev = rc.pos_dev;
            KR_TRY(model_gemm(rc, G_QKV, l, T, u + b * td, td, e, b, 1, st));
            {
                LaunchScope scope(h, KRAKEN_PROF_ATTENTION, st);
                DecodeAttnParams dp;
                dp.q = q + b * td; dp.q_gstride = td;
                dp.k_cache = e.k_cache; dp.v_cache = e.v_cache;
                dp.cache_gstride = 2 * cache_kv; dp.cache_bstride = cache_b;
                dp.groups = 1; dp.batch = rc.batch; dp.n_keys = rc.pos0 + 1; dp.n_head = H; dp.head_dim = hd;
                dp.n_kv_head = Hkv;
                dp.max_pos = c.max_pos;
                dp.pos_dev = rc.pos_dev;
                dp.splits = splits;
                dp.partials = at<float>(h, h->lay.dec_part) + b * part_b;
                dp.out = o + b * td; dp.out_gstride = td;
                h->launches[KRAKEN_PROF_ATTENTION] += dp.splits > 1 ? 1 : 0;
                KR_TRY(launch_attention_decode(dp, st));
            }
            e = epi_zero();
            e.kind = KRAKEN_EPI_RESID_F32;
            e.out_f32 = a + b * td; e.out_f32_gstride = td; e.ld_out_f32 = d;
            e.resid = xin; e.resid_gstride = 0; e.ld_resid = d;
            KR_TRY(model_gemm(rc, G_PROJ, l, T, o + b * td, td, e, b, 1, st));
            // LayerNorm-2 sums the previous layer's outputs of every branch
            if (l > 0 && !c.no_combine && !c.parallel_ffn)
                for (int j = 0; j < N; ++j)
                    if (j != b) KR_CU(cudaStreamWaitEvent(st, h->ev_down[(l - 1) & 1][j], 0));
            if (!c.parallel_ffn) {
                LaunchScope scope(h, KRAKEN_PROF_LAYERNORM, st);
                KR_TRY(launch_layernorm(a + b * td, 0, (l == 0 && !c.no_combine) ? x0 : nullptr,
                                        (const uint16_t *)h->w.ln2_g + ln_off + (long long)b * d,
                                        h->w.ln2_b ? (const uint16_t *)h->w.ln2_b + ln_off + (long long)b * d : nullptr,
                                        1, T, d, c.ln_eps, u + b * td, st,
                                        (l == 0 || c.no_combine) ? nullptr : xprev, td, N));
            }
            e = epi_zero();
            e.kind = KRAKEN_EPI_GELU_BF16;
            e.out_bf16 = gb + b * (long long)T * F; e.out_bf16_gstride = (long long)T * F; e.ld_out_bf16 = F;
            e.gelu_tanh = c.gelu_tanh;
            KR_TRY(model_gemm(rc, G_UP, l, T, u + b * td, td, e, b, 1, st));
            e = epi_zero();
            e.kind = KRAKEN_EPI_RESID_F32;
            e.out_f32 = xout + b * td; e.out_f32_gstride = td; e.ld_out_f32 = d;
            e.resid = a + b * td; e.resid_gstride = td; e.ld_resid = d;
            KR_TRY(model_gemm(rc, G_DOWN, l, T, gb + b * (long long)T * F, (long long)T * F, e, b, 1, st));
            KR_CU(cudaEventRecord(h->ev_down[l & 1][b], st));
        }
    }
    for (int b = 1; b < N; ++b) {
        KR_CU(cudaEventRecord(h->ev_join[b], h->br_stream[b]));
        KR_CU(cudaStreamWaitEvent(rc.st, h->ev_join[b], 0));
    }
#undef KR_CU
    h->last_rows = T;
    return KRAKEN_OK;
}

void advance_lengths(kraken_handle *h) {
    h->cur_len += 1;
    for (int &v : h->seq_len) v += 1;
}

// The next position of every sequence lives in device memory (the decode graph reads it there).
__global__ void set_pos_kernel(int *pos, int value, int batch) {
    pdl_wait();
    for (int b = threadIdx.x; b < batch; b += blockDim.x) pos[b] = value;
}
__global__ void advance_pos_kernel(int *pos, int batch) {
    pdl_wait();
    for (int b = threadIdx.x; b < batch; b += blockDim.x) pos[b] += 1;
}

__global__ void make_rows_kernel(int32_t *rows, int n, int mul, int add) {
    pdl_wait();
    pdl_trigger();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) rows[i] = i * mul + add;
}

// W_concat, final LayerNorm and the tied unembedding for n_rows token rows (device index list).
// W_concat over the chosen rows of the last layer's outputs: z [n_rows, d] fp32.
int tail_concat(const RunCtx &rc, const int32_t *d_rows, int n_rows, float *z) {
    kraken_handle *h = rc.h;
    const kraken_config &c = h->cfg;
    const int d = c.d_model, N = c.n_branch;
    const long long td = (long long)h->last_rows * d;
    float *x = at<float>(h, h->lay.x);
    uint16_t *cat = at<uint16_t>(h, h->lay.u);
    {
        LaunchScope scope(h, KRAKEN_PROF_TAIL, rc.st);
        if (short_last_of(rc))   // the last layer left one row per sequence, in sequence order: exactly the rows asked for
            KR_TRY(launch_gather_concat(at<float>(h, h->lay.last_x), (long long)n_rows * d, N, d, nullptr, n_rows, cat, rc.st));
        else
            KR_TRY(launch_gather_concat(x, td, N, d, d_rows, n_rows, cat, rc.st));
    }
    EpiParams e = epi_zero();
    e.kind = KRAKEN_EPI_F32;
    e.out_f32 = z; e.ld_out_f32 = d;
    return model_gemm(rc, G_CONCAT, 0, n_rows, cat, 0, e);
}

// Final LayerNorm (if configured) and the tied unembedding of z [n_rows, d].
int tail_head(const RunCtx &rc, const float *z, int n_rows, float *d_logits) {
    kraken_handle *h = rc.h;
    const kraken_config &c = h->cfg;
    const int d = c.d_model;
    uint16_t *zf = at<uint16_t>(h, h->lay.q);
    {
        LaunchScope scope(h, KRAKEN_PROF_TAIL, rc.st);
        if (c.final_ln) {
            KR_TRY(launch_layernorm(z, 0, nullptr, (const uint16_t *)h->w.lnf_g, (const uint16_t *)h->w.lnf_b, 1,
                                    n_rows, d, c.ln_eps, zf, rc.st));
        } else {
            KR_TRY(launch_f32_to_bf16(z, zf, (long long)n_rows * d, rc.st));
        }
    }
    EpiParams e = epi_zero();
    e.kind = KRAKEN_EPI_F32;
    e.out_f32 = d_logits; e.ld_out_f32 = c.vocab;
    return model_gemm(rc, G_HEAD, 0, n_rows, zf, 0, e);
}

int run_tail(const RunCtx &rc, const int32_t *d_rows, int n_rows, float *d_logits) {
    // z normally borrows the cross-branch sum's buffer; after a short last layer that sum (and q) must survive, in
    // case kraken_logits_rows runs the layer on every row later, so z then goes where the gathered y rows were
    float *z = short_last_of(rc) ? at<float>(rc.h, rc.h->lay.last_y) : at<float>(rc.h, rc.h->lay.s);
    KR_TRY(tail_concat(rc, d_rows, n_rows, z));
    return tail_head(rc, z, n_rows, d_logits);
}

// The kernel sequence of one prefill on stream st.
int prefill_body(kraken_handle *h, cudaStream_t st, const int32_t *d_tokens, int batch, int seqlen, float *d_logits,
                 bool all_logits) {
    RunCtx rc{h, st, batch, seqlen, 0, batch * seqlen, nullptr, 0};
    int32_t *rows = at<int32_t>(h, h->lay.rows);
    const int n_rows = all_logits ? batch * seqlen : batch;
    h->launches[KRAKEN_PROF_TAIL]++;
    make_rows_kernel<<<(n_rows + 255) / 256, 256, 0, st>>>(rows, n_rows, all_logits ? 1 : seqlen,
                                                           all_logits ? 0 : seqlen - 1);
    if (cudaGetLastError() != cudaSuccess) return KRAKEN_ECUDA;
    rc.last_only = !all_logits && tuning(KRAKEN_TUNE_LAST_LAYER) != 1;
    rc.last_rows = rows;
    KR_TRY(run_layers(rc, d_tokens));
    set_pos_kernel<<<1, 64, 0, st>>>(at<int>(h, h->lay.pos_arr), seqlen, batch);
    return run_tail(rc, rows, n_rows, d_logits);
}

int prefill_common(kraken_handle *h, const int32_t *d_tokens, int batch, int seqlen, float *d_logits, void *stream,
                   bool all_logits) {
    if (!h || !d_tokens || !d_logits || batch < 1 || seqlen < 1) return KRAKEN_EINVAL;
    if (batch > h->cfg.max_batch || seqlen > h->cfg.max_pos) return KRAKEN_ECAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    h->last_stream = st;
    const bool same = h->pre_tokens == d_tokens && h->pre_logits == d_logits && h->pre_batch == batch &&
                      h->pre_seqlen == seqlen && h->pre_all == (all_logits ? 1 : 0);
    if (!same) {
        if (h->pre_graph) cudaGraphExecDestroy(h->pre_graph);
        h->pre_graph = nullptr;
        h->pre_tokens = d_tokens;
        h->pre_logits = d_logits;
        h->pre_batch = batch;
        h->pre_seqlen = seqlen;
        h->pre_all = all_logits ? 1 : 0;
        h->pre_seen = 0;
    }
    {
        RunCtx probe{h, st, batch, seqlen, 0, batch * seqlen, nullptr, 0};
        probe.last_only = !all_logits && tuning(KRAKEN_TUNE_LAST_LAYER) != 1;
        probe.last_rows = at<int32_t>(h, h->lay.rows);
        h->x_partial = short_last_of(probe);
    }
    bool done = false;
    if (h->use_graph && !h->prof_on && h->pre_seen >= 1) {
        // second and later calls with the same shape and buffers: capture once, then replay
        if (!h->pre_graph) {
            long long before[KRAKEN_PROF_COUNT];
            for (int i = 0; i < KRAKEN_PROF_COUNT; ++i) before[i] = h->launches[i];
            if (!h->cap_stream)
                KR_TRY(cuda_check(cudaStreamCreateWithFlags(&h->cap_stream, cudaStreamNonBlocking),
                                  "prefill: capture stream"));
            KR_TRY(cuda_check(cudaStreamBeginCapture(h->cap_stream, cudaStreamCaptureModeThreadLocal),
                              "prefill: begin capture"));
            const int rc_body = prefill_body(h, h->cap_stream, d_tokens, batch, seqlen, d_logits, all_logits);
            cudaGraph_t graph = nullptr;
            cudaError_t ce = cudaStreamEndCapture(h->cap_stream, &graph);
            for (int i = 0; i < KRAKEN_PROF_COUNT; ++i) {
                h->pre_graph_launches[i] = h->launches[i] - before[i];
                h->launches[i] = before[i];
            }
            if (!rc_body && ce == cudaSuccess && graph)
                ce = cudaGraphInstantiate(&h->pre_graph, graph, 0);
            else
                ce = cudaErrorUnknown;
            if (graph) cudaGraphDestroy(graph);
            if (ce != cudaSuccess) {
                h->pre_graph = nullptr;
                h->use_graph = false;             // eager from now on for this handle
                cudaGetLastError();
            }
        }
        if (h->pre_graph) {
            KR_TRY(cuda_check(cudaGraphLaunch(h->pre_graph, st), "prefill: graph launch"));
            for (int i = 0; i < KRAKEN_PROF_COUNT; ++i) h->launches[i] += h->pre_graph_launches[i];
            h->last_rows = batch * seqlen;
            done = true;
        }
    }
    if (!done) KR_TRY(prefill_body(h, st, d_tokens, batch, seqlen, d_logits, all_logits));
    h->pre_seen++;
    h->cur_len = seqlen;
    h->batch = batch;
    h->last_seqlen = seqlen;
    h->seq_len.assign(batch, seqlen);
    h->ragged = false;
    return KRAKEN_OK;
}

// Packed prefill: the sequences of the batch have their own lengths and their tokens follow each other
// without padding.  Everything that works on token rows (LayerNorms, GEMMs) sees one [sum of lengths, d]
// tensor; the embedding and the K/V scatter take a row's sequence and position from two small tables;
// attention runs once per sequence on that sequence's rows.
int prefill_packed(kraken_handle *h, const int32_t *d_tokens, const int32_t *h_seq_lens, int batch, float *d_logits,
                   void *stream) {
    if (!h || !d_tokens || !h_seq_lens || !d_logits || batch < 1) return KRAKEN_EINVAL;
    h->x_partial = false;
    if (batch > h->cfg.max_batch) return KRAKEN_ECAPACITY;
    long long total = 0;
    int longest = 0;
    for (int b = 0; b < batch; ++b) {
        if (h_seq_lens[b] < 1) return KRAKEN_EINVAL;
        if (h_seq_lens[b] > h->cfg.max_pos) return KRAKEN_ECAPACITY;
        total += h_seq_lens[b];
        longest = h_seq_lens[b] > longest ? h_seq_lens[b] : longest;
    }
    if (total > (long long)h->cfg.max_batch * h->cfg.max_pos) return KRAKEN_ECAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    h->last_stream = st;
    if (h->pre_graph) cudaGraphExecDestroy(h->pre_graph);     // the cached prefill graph belongs to another shape
    h->pre_graph = nullptr;
    h->pre_tokens = nullptr;
    h->pre_seen = 0;
    const int T = static_cast<int>(total);
    h->seq_len.assign(h_seq_lens, h_seq_lens + batch);
    h->host_row_seq.resize(T);
    h->host_row_pos.resize(T);
    h->host_rows.resize(batch);
    int r = 0;
    for (int b = 0; b < batch; ++b) {
        for (int t = 0; t < h_seq_lens[b]; ++t, ++r) {
            h->host_row_seq[r] = b;
            h->host_row_pos[r] = t;
        }
        h->host_rows[b] = r - 1;                              // last position of the sequence
    }
    int *d_row_seq = at<int>(h, h->lay.row_seq), *d_row_pos = at<int>(h, h->lay.row_pos);
    int32_t *rows = at<int32_t>(h, h->lay.rows);
    int *d_pos = at<int>(h, h->lay.pos_arr);
    if (cudaMemcpyAsync(d_row_seq, h->host_row_seq.data(), (size_t)T * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(d_row_pos, h->host_row_pos.data(), (size_t)T * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(rows, h->host_rows.data(), (size_t)batch * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(d_pos, h->seq_len.data(), (size_t)batch * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return cuda_check(cudaGetLastError(), "packed prefill: table upload");
    RunCtx rc{h, st, batch, longest, 0, T, nullptr, 0, true, d_row_seq, d_row_pos};
    // last-position logits only: the last layer runs on one row per sequence past its qkv GEMM (RunCtx::last_only)
    h->host_len_m1.resize(batch);
    for (int b = 0; b < batch; ++b) h->host_len_m1[b] = h_seq_lens[b] - 1;
    int *d_len_m1 = at<int>(h, h->lay.last_len);
    if (cudaMemcpyAsync(d_len_m1, h->host_len_m1.data(), (size_t)batch * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return cuda_check(cudaGetLastError(), "packed prefill: table upload");
    rc.last_only = tuning(KRAKEN_TUNE_LAST_LAYER) != 1;
    rc.last_rows = rows;
    rc.last_len_m1 = d_len_m1;
    KR_TRY(run_layers(rc, d_tokens));
    KR_TRY(run_tail(rc, rows, batch, d_logits));
    h->x_partial = short_last_of(rc);
    h->cur_len = longest;
    h->batch = batch;
    h->last_seqlen = longest;
    h->ragged = true;
    return KRAKEN_OK;
}

}  // namespace

extern "C" {

int kraken_query_sizes(const kraken_config *cfg, size_t *kv_bytes, size_t *scratch_bytes) {
    int rc = check_config(cfg);
    if (rc) return rc;
    if (!kv_bytes || !scratch_bytes) return KRAKEN_EINVAL;
    *kv_bytes = kv_bytes_of(cfg);
    *scratch_bytes = layout_of(cfg).total;
    return KRAKEN_OK;
}

int kraken_create(const kraken_config *cfg, const kraken_weights *w, void *d_kv, size_t kv_bytes, void *d_scratch,
                  size_t scratch_bytes, kraken_handle **out) {
    int rc = check_config(cfg);
    if (rc) return rc;
    if (!w || !d_kv || !d_scratch || !out) return KRAKEN_EINVAL;
    if (!w->wte || !w->wpe || !w->ln1_g || !w->w_qkv || !w->w_proj || !w->ln2_g || !w->w_up || !w->w_down ||
        !w->w_concat || (cfg->final_ln && !w->lnf_g))
        return KRAKEN_EINVAL;
    if ((reinterpret_cast<uintptr_t>(d_kv) & (ALIGN - 1)) || (reinterpret_cast<uintptr_t>(d_scratch) & (ALIGN - 1)))
        return KRAKEN_EINVAL;
    Layout lay = layout_of(cfg);
    if (kv_bytes < kv_bytes_of(cfg) || scratch_bytes < lay.total) return KRAKEN_ECAPACITY;
    kraken_handle *h = new (std::nothrow) kraken_handle();
    if (!h) return KRAKEN_EINVAL;
    h->cfg = *cfg;
    h->w = *w;
    h->kv = static_cast<uint8_t *>(d_kv);
    h->scratch = static_cast<uint8_t *>(d_scratch);
    h->lay = lay;
    h->cur_len = 0;
    h->batch = 0;
    h->last_seqlen = 0;
    h->last_rows = 0;
    h->last_stream = nullptr;
    // the two environment switches of a handle are read here, once; nothing on the launch path reads the environment
    h->one_chain = env_flag("KRAKEN_DECODE_ONE_CHAIN");
    h->prof_on = false;
    h->dec_graph = nullptr;
    h->pre_graph = nullptr;
    h->pre_tokens = h->pre_logits = nullptr;
    h->pre_batch = h->pre_seqlen = h->pre_all = h->pre_seen = 0;
    h->cap_stream = nullptr;
    h->br_ready = false;
    h->ragged = false;
    h->stage_layer_done = -1;
    h->stage_decode = false;
    h->dec_graph_batch = 0;
    h->dec_eager_steps = 0;
    h->use_graph = !env_flag("KRAKEN_NO_GRAPH");
    h->ev_used = 0;
    for (int i = 0; i < KRAKEN_PROF_COUNT; ++i) h->launches[i] = 0;
    for (int i = 0; i < G_COUNT; ++i) {
        h->tmB_bn[i] = 0;
        h->tmA_key[i] = {nullptr, 0, 0, 0};
    }
    if (cudaMemset(h->scratch + lay.ln_cnt, 0, lay.ln_cnt_bytes) != cudaSuccess ||
        cudaMemset(h->scratch + lay.status, 0, 256) != cudaSuccess) {
        delete h;
        return KRAKEN_ECUDA;
    }
    *out = h;
    return KRAKEN_OK;
}

int kraken_prefill(kraken_handle *h, const int32_t *d_tokens, int32_t batch, int32_t seqlen, float *d_logits,
                   void *stream) {
    return prefill_common(h, d_tokens, batch, seqlen, d_logits, stream, false);
}

int kraken_prefill_packed(kraken_handle *h, const int32_t *d_tokens, const int32_t *h_seq_lens, int32_t batch,
                          float *d_logits, void *stream) {
    return prefill_packed(h, d_tokens, h_seq_lens, batch, d_logits, stream);
}

// ---- branch-parallel deployment: the path in pieces (see kraken.h)

// Run context of one piece: a prefill of batch x last_seqlen tokens at position 0, or a decode step whose
// positions come from the device array.
static RunCtx stage_ctx(kraken_handle *h, cudaStream_t st, int stage, int layer, const float *y) {
    if (h->stage_decode)
        return RunCtx{h, st, h->batch, 1, h->cur_len, h->batch, at<int>(h, h->lay.pos_arr), h->cfg.max_pos,
                      false, nullptr, nullptr, stage, layer, y};
    return RunCtx{h, st, h->batch, h->last_seqlen, 0, h->batch * h->last_seqlen, nullptr, 0,
                  false, nullptr, nullptr, stage, layer, y};
}

int kraken_stage_begin(kraken_handle *h, const int32_t *d_tokens, int32_t batch, int32_t seqlen, void *stream) {
    if (!h || !d_tokens || batch < 1 || seqlen < 1) return KRAKEN_EINVAL;
    h->x_partial = false;   // whatever runs now leaves every row's outputs, or none that kraken_logits_rows may read
    if (batch > h->cfg.max_batch || seqlen > h->cfg.max_pos) return KRAKEN_ECAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    h->last_stream = st;
    if (h->pre_graph) cudaGraphExecDestroy(h->pre_graph);
    h->pre_graph = nullptr;
    h->pre_tokens = nullptr;
    h->pre_seen = 0;
    h->cur_len = 0;                       // nothing is cached until kraken_stage_head has run
    h->batch = batch;
    h->last_seqlen = seqlen;
    h->stage_layer_done = -1;
    h->stage_decode = false;
    RunCtx rc{h, st, batch, seqlen, 0, batch * seqlen, nullptr, 0, false, nullptr, nullptr, STAGE_EMBED, 0, nullptr};
    KR_TRY(run_layers(rc, d_tokens));
    h->last_rows = batch * seqlen;
    return KRAKEN_OK;
}

int kraken_stage_begin_decode(kraken_handle *h, const int32_t *d_tokens, int32_t batch, void *stream) {
    if (!h || !d_tokens || batch < 1) return KRAKEN_EINVAL;
    h->x_partial = false;   // whatever runs now leaves every row's outputs, or none that kraken_logits_rows may read
    if (h->cur_len < 1 || batch != h->batch) return KRAKEN_ESTATE;
    if (h->cur_len + 1 > h->cfg.max_pos) return KRAKEN_ECAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    h->last_stream = st;
    h->last_seqlen = 1;
    h->stage_layer_done = -1;
    h->stage_decode = true;
    RunCtx rc = stage_ctx(h, st, STAGE_EMBED, 0, nullptr);
    KR_TRY(run_layers(rc, d_tokens));
    h->last_rows = batch;
    return KRAKEN_OK;
}

int kraken_stage_attention(kraken_handle *h, int32_t layer, void *stream) {
    if (!h || layer < 0 || layer >= h->cfg.n_layer) return KRAKEN_EINVAL;
    if (h->batch < 1 || h->last_seqlen < 1 || layer != h->stage_layer_done + 1) return KRAKEN_ESTATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    h->last_stream = st;
    RunCtx rc = stage_ctx(h, st, STAGE_ATTN, layer, nullptr);
    return run_layers(rc, nullptr);
}

int kraken_stage_ffn(kraken_handle *h, int32_t layer, const float *d_y, void *stream) {
    if (!h || layer < 0 || layer >= h->cfg.n_layer || !d_y) return KRAKEN_EINVAL;
    if (h->batch < 1 || h->last_seqlen < 1 || layer != h->stage_layer_done + 1) return KRAKEN_ESTATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    h->last_stream = st;
    RunCtx rc = stage_ctx(h, st, STAGE_FFN, layer, d_y);
    KR_TRY(run_layers(rc, nullptr));
    h->stage_layer_done = layer;
    return KRAKEN_OK;
}

int kraken_stage_buffers(kraken_handle *h, float **d_x0, float **d_local_sum) {
    if (!h || !d_x0 || !d_local_sum) return KRAKEN_EINVAL;
    *d_x0 = at<float>(h, h->lay.x0);
    *d_local_sum = at<float>(h, h->lay.s);
    return KRAKEN_OK;
}

int kraken_stage_concat(kraken_handle *h, float *d_z, void *stream) {
    if (!h || !d_z) return KRAKEN_EINVAL;
    if (h->batch < 1 || h->stage_layer_done != h->cfg.n_layer - 1) return KRAKEN_ESTATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    h->last_stream = st;
    RunCtx rc = stage_ctx(h, st, STAGE_ALL, 0, nullptr);
    int32_t *rows = at<int32_t>(h, h->lay.rows);
    h->launches[KRAKEN_PROF_TAIL]++;
    make_rows_kernel<<<(h->batch + 255) / 256, 256, 0, st>>>(rows, h->batch, h->last_seqlen, h->last_seqlen - 1);
    if (cudaGetLastError() != cudaSuccess) return KRAKEN_ECUDA;
    return tail_concat(rc, rows, h->batch, d_z);
}

int kraken_stage_head(kraken_handle *h, const float *d_z, float *d_logits, void *stream) {
    if (!h || !d_z || !d_logits) return KRAKEN_EINVAL;
    if (h->batch < 1 || h->stage_layer_done != h->cfg.n_layer - 1) return KRAKEN_ESTATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    h->last_stream = st;
    RunCtx rc = stage_ctx(h, st, STAGE_ALL, 0, nullptr);
    KR_TRY(tail_head(rc, d_z, h->batch, d_logits));
    h->stage_layer_done = -1;
    if (h->stage_decode) {
        advance_pos_kernel<<<1, 64, 0, st>>>(at<int>(h, h->lay.pos_arr), h->batch);
        advance_lengths(h);
    } else {
        set_pos_kernel<<<1, 64, 0, st>>>(at<int>(h, h->lay.pos_arr), h->last_seqlen, h->batch);
        h->cur_len = h->last_seqlen;
        h->seq_len.assign(h->batch, h->last_seqlen);
        h->ragged = false;
    }
    return cuda_check(cudaGetLastError(), "stage head: position update");
}

int kraken_seq_lens(kraken_handle *h, int32_t *h_seq_lens, int32_t batch) {
    if (!h || !h_seq_lens || batch < 1) return KRAKEN_EINVAL;
    if (batch != h->batch || (int)h->seq_len.size() != batch) return KRAKEN_ESTATE;
    for (int b = 0; b < batch; ++b) h_seq_lens[b] = h->seq_len[b];
    return KRAKEN_OK;
}

int kraken_prefill_all_logits(kraken_handle *h, const int32_t *d_tokens, int32_t batch, int32_t seqlen,
                              float *d_logits, void *stream) {
    return prefill_common(h, d_tokens, batch, seqlen, d_logits, stream, true);
}

int kraken_prefill_host(kraken_handle *h, const int32_t *h_tokens, int32_t batch, int32_t seqlen, float *h_logits,
                        void *stream) {
    if (!h || !h_tokens || !h_logits || batch < 1 || seqlen < 1) return KRAKEN_EINVAL;
    if (batch > h->cfg.max_batch || seqlen > h->cfg.max_pos) return KRAKEN_ECAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t *d_tok = at<int32_t>(h, h->lay.tokens);
    float *d_log = at<float>(h, h->lay.logits);
    if (cudaMemcpyAsync(d_tok, h_tokens, (size_t)batch * seqlen * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return KRAKEN_ECUDA;
    KR_TRY(prefill_common(h, d_tok, batch, seqlen, d_log, stream, false));
    if (cudaMemcpyAsync(h_logits, d_log, (size_t)batch * h->cfg.vocab * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return KRAKEN_ECUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? KRAKEN_OK : KRAKEN_ECUDA;
}

int kraken_logits_rows(kraken_handle *h, const int32_t *h_rows, int32_t n_rows, float *d_logits, void *stream) {
    if (!h || !h_rows || !d_logits || n_rows < 1) return KRAKEN_EINVAL;
    if (h->last_rows < 1) return KRAKEN_ESTATE;
    if ((long long)n_rows > (long long)h->cfg.max_batch * h->cfg.max_pos) return KRAKEN_ECAPACITY;
    for (int i = 0; i < n_rows; ++i)
        if (h_rows[i] < 0 || h_rows[i] >= h->last_rows) return KRAKEN_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    RunCtx rc{h, st, h->batch, h->last_seqlen, 0, h->last_rows, nullptr, 0};
    h->last_stream = st;
    if (h->x_partial) {
        // the prefill ran its last layer for the last positions only: run that layer on every row now (its inputs,
        // the previous layer's outputs and their sum, are untouched; K and V are written again with the same values)
        RunCtx full = rc;
        if (h->ragged) {
            full.packed = true;
            full.row_seq = at<int>(h, h->lay.row_seq);
            full.row_pos = at<int>(h, h->lay.row_pos);
        }
        full.only_layer = h->cfg.n_layer - 1;
        KR_TRY(run_layers(full, nullptr));
        h->x_partial = false;
    }
    int32_t *rows = at<int32_t>(h, h->lay.rows);
    if (cudaMemcpyAsync(rows, h_rows, (size_t)n_rows * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return KRAKEN_ECUDA;
    return run_tail(rc, rows, n_rows, d_logits);
}

namespace {

// Whether decode steps of this handle run the branches as concurrent chains.
bool decode_chains(const kraken_handle *h) {
    return h->cfg.n_branch >= 2 && h->cfg.n_branch <= MAX_CHAINS && !h->one_chain;
}

// The kernel sequence of one decode step; with from_dev the position is read from device memory.
int decode_body(kraken_handle *h, cudaStream_t st, const int32_t *d_tokens, int batch, float *d_logits,
                bool from_dev) {
    // positions always come from the device array: the sequences of a batch may differ in length
    int *d_pos = at<int>(h, h->lay.pos_arr);
    (void)from_dev;
    RunCtx rc{h, st, batch, 1, h->cur_len, batch, d_pos, h->cfg.max_pos};
    // per-kernel timing wants the kernels one after the other, so profiled steps keep all branches in one chain
    if (decode_chains(h) && !h->prof_on) {
        KR_TRY(run_layers_decode_branches(rc, d_tokens));
    } else {
        KR_TRY(run_layers(rc, d_tokens));
    }
    h->last_seqlen = 1;
    int32_t *rows = at<int32_t>(h, h->lay.rows);
    h->launches[KRAKEN_PROF_TAIL]++;
    make_rows_kernel<<<(batch + 255) / 256, 256, 0, st>>>(rows, batch, 1, 0);
    if (cudaGetLastError() != cudaSuccess) return KRAKEN_ECUDA;
    KR_TRY(run_tail(rc, rows, batch, d_logits));
    advance_pos_kernel<<<1, 64, 0, st>>>(d_pos, batch);
    return cuda_check(cudaGetLastError(), "decode: position update");
}

}  // namespace

int kraken_decode_step(kraken_handle *h, const int32_t *d_tokens, int32_t batch, float *d_logits, void *stream) {
    if (!h || !d_tokens || !d_logits || batch < 1) return KRAKEN_EINVAL;
    h->x_partial = false;   // whatever runs now leaves every row's outputs, or none that kraken_logits_rows may read
    if (h->cur_len < 1 || batch != h->batch) return KRAKEN_ESTATE;
    if (h->cur_len + 1 > h->cfg.max_pos) return KRAKEN_ECAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    h->last_stream = st;
    if (decode_chains(h)) KR_TRY(branch_streams(h));   // created outside any capture
    if (h->dec_graph_batch != batch) {            // a new batch size: forget the old graph, warm up again
        if (h->dec_graph) cudaGraphExecDestroy(h->dec_graph);
        h->dec_graph = nullptr;
        h->dec_graph_batch = batch;
        h->dec_eager_steps = 0;
    }
    if (!h->use_graph || h->prof_on || h->dec_eager_steps < 1) {
        // eager step (also the first step of a batch size: it performs every one-time set-up call,
        // none of which may happen inside a stream capture)
        KR_TRY(decode_body(h, st, d_tokens, batch, d_logits, false));
        h->dec_eager_steps++;
        advance_lengths(h);
        return KRAKEN_OK;
    }
    int32_t *s_tok = at<int32_t>(h, h->lay.tokens);
    float *s_log = at<float>(h, h->lay.logits);
    if (d_tokens != s_tok)
        KR_TRY(cuda_check(cudaMemcpyAsync(s_tok, d_tokens, (size_t)batch * 4, cudaMemcpyDeviceToDevice, st),
                          "decode: token staging"));
    if (!h->dec_graph) {
        long long before[KRAKEN_PROF_COUNT];
        for (int i = 0; i < KRAKEN_PROF_COUNT; ++i) before[i] = h->launches[i];
        if (!h->cap_stream)
            KR_TRY(cuda_check(cudaStreamCreateWithFlags(&h->cap_stream, cudaStreamNonBlocking), "decode: capture stream"));
        KR_TRY(cuda_check(cudaStreamBeginCapture(h->cap_stream, cudaStreamCaptureModeThreadLocal),
                          "decode: begin capture"));
        const int saved_len = h->cur_len, saved_rows = h->last_rows;
        int rc_body = decode_body(h, h->cap_stream, s_tok, batch, s_log, true);
        cudaGraph_t graph = nullptr;
        cudaError_t ce = cudaStreamEndCapture(h->cap_stream, &graph);
        h->cur_len = saved_len;
        h->last_rows = saved_rows;
        for (int i = 0; i < KRAKEN_PROF_COUNT; ++i) {
            h->dec_graph_launches[i] = h->launches[i] - before[i];
            h->launches[i] = before[i];
        }
        if (rc_body || ce != cudaSuccess || !graph) {
            if (graph) cudaGraphDestroy(graph);
            cudaGetLastError();
            h->use_graph = false;                 // fall back to eager steps for this handle
            KR_TRY(decode_body(h, st, d_tokens, batch, d_logits, false));
            advance_lengths(h);
            return KRAKEN_OK;
        }
        ce = cudaGraphInstantiate(&h->dec_graph, graph, 0);
        cudaGraphDestroy(graph);
        if (ce != cudaSuccess) {
            h->dec_graph = nullptr;
            h->use_graph = false;
            cudaGetLastError();
            KR_TRY(decode_body(h, st, d_tokens, batch, d_logits, false));
            advance_lengths(h);
            return KRAKEN_OK;
        }
    }
    KR_TRY(cuda_check(cudaGraphLaunch(h->dec_graph, st), "decode: graph launch"));
    for (int i = 0; i < KRAKEN_PROF_COUNT; ++i) h->launches[i] += h->dec_graph_launches[i];
    h->last_rows = batch;
    h->last_seqlen = 1;
    if (d_logits != s_log)
        KR_TRY(cuda_check(cudaMemcpyAsync(d_logits, s_log, (size_t)batch * h->cfg.vocab * 4,
                                          cudaMemcpyDeviceToDevice, st), "decode: logits staging"));
    advance_lengths(h);
    return KRAKEN_OK;
}

int kraken_decode_step_host(kraken_handle *h, const int32_t *h_tokens, int32_t batch, float *h_logits, void *stream) {
    if (!h || !h_tokens || !h_logits || batch < 1) return KRAKEN_EINVAL;
    if (batch > h->cfg.max_batch) return KRAKEN_ECAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t *d_tok = at<int32_t>(h, h->lay.tokens);
    float *d_log = at<float>(h, h->lay.logits);
    if (cudaMemcpyAsync(d_tok, h_tokens, (size_t)batch * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return KRAKEN_ECUDA;
    KR_TRY(kraken_decode_step(h, d_tok, batch, d_log, stream));
    if (cudaMemcpyAsync(h_logits, d_log, (size_t)batch * h->cfg.vocab * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return KRAKEN_ECUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? KRAKEN_OK : KRAKEN_ECUDA;
}

int kraken_kv_view(kraken_handle *h, int32_t layer, int32_t branch, int32_t which, const void **ptr,
                   int64_t strides[4]) {
    if (!h || !ptr || !strides) return KRAKEN_EINVAL;
    const kraken_config &c = h->cfg;
    if (layer < 0 || layer >= c.n_layer || branch < 0 || branch >= c.n_branch || which < 0 || which > 1)
        return KRAKEN_EINVAL;
    const int hd = c.d_model / c.n_head;
    const long long cache_b = (long long)kv_heads_of(c) * c.max_pos * hd, cache_kv = (long long)c.max_batch * cache_b;
    *ptr = reinterpret_cast<uint16_t *>(h->kv) + (((long long)layer * c.n_branch + branch) * 2 + which) * cache_kv;
    strides[0] = cache_b;
    strides[1] = (long long)c.max_pos * hd;
    strides[2] = hd;
    strides[3] = 1;
    return KRAKEN_OK;
}

int kraken_device_status(kraken_handle *h, uint32_t *flags) {
    if (!h || !flags) return KRAKEN_EINVAL;
    if (cudaStreamSynchronize(h->last_stream) != cudaSuccess) return KRAKEN_ECUDA;
    if (cudaMemcpy(flags, h->scratch + h->lay.status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return KRAKEN_ECUDA;
    return KRAKEN_OK;
}

int kraken_cur_len(kraken_handle *h, int32_t *cur_len) {
    if (!h || !cur_len) return KRAKEN_EINVAL;
    *cur_len = h->cur_len;
    return KRAKEN_OK;
}

int kraken_reset(kraken_handle *h) {
    if (!h) return KRAKEN_EINVAL;
    h->x_partial = false;   // whatever runs now leaves every row's outputs, or none that kraken_logits_rows may read
    if (cudaStreamSynchronize(h->last_stream) != cudaSuccess) return KRAKEN_ECUDA;
    if (cudaMemset(h->scratch + h->lay.status, 0, 256) != cudaSuccess) return KRAKEN_ECUDA;
    if (cudaMemset(h->scratch + h->lay.ln_cnt, 0, h->lay.ln_cnt_bytes) != cudaSuccess) return KRAKEN_ECUDA;
    h->cur_len = 0;
    h->batch = 0;
    h->last_rows = 0;
    h->last_seqlen = 0;
    h->seq_len.clear();
    h->ragged = false;
    return KRAKEN_OK;
}

void kraken_destroy(kraken_handle *h) {
    if (!h) return;
    for (cudaEvent_t e : h->ev_pool) cudaEventDestroy(e);
    if (h->dec_graph) cudaGraphExecDestroy(h->dec_graph);
    if (h->pre_graph) cudaGraphExecDestroy(h->pre_graph);
    if (h->cap_stream) cudaStreamDestroy(h->cap_stream);
    if (h->br_ready) {
        for (int b = 0; b < MAX_CHAINS; ++b) {
            cudaStreamDestroy(h->br_stream[b]);
            cudaEventDestroy(h->ev_join[b]);
            cudaEventDestroy(h->ev_down[0][b]);
            cudaEventDestroy(h->ev_down[1][b]);
        }
        cudaEventDestroy(h->ev_fork);
    }
    delete h;
}

int kraken_profile_enable(kraken_handle *h, int32_t on) {
    if (!h) return KRAKEN_EINVAL;
    h->prof_on = on != 0;
    return KRAKEN_OK;
}

int kraken_profile_read(kraken_handle *h, double *ms, int64_t *launches) {
    if (!h || !ms || !launches) return KRAKEN_EINVAL;
    if (cudaStreamSynchronize(h->last_stream) != cudaSuccess) return KRAKEN_ECUDA;
    for (int i = 0; i < KRAKEN_PROF_COUNT; ++i) {
        ms[i] = 0.0;
        launches[i] = h->launches[i];
        h->launches[i] = 0;
    }
    for (const auto &sp : h->spans) {
        float t = 0.f;
        if (cudaEventElapsedTime(&t, h->ev_pool[sp.e0], h->ev_pool[sp.e1]) != cudaSuccess) return KRAKEN_ECUDA;
        ms[sp.cat] += t;
    }
    h->spans.clear();
    h->ev_used = 0;
    return KRAKEN_OK;
}

const char *kraken_last_cuda_error(void) { return last_cuda_error(); }

int kraken_tuning_set(int32_t key, int32_t value) { return set_tuning(key, value); }

int kraken_storage_dtype(void) { return KRAKEN_F16 ? 1 : 0; }

const char *kraken_strerror(int status) {
    switch (status) {
        case KRAKEN_OK: return "ok";
        case KRAKEN_EINVAL: return "invalid argument";
        case KRAKEN_EUNSUPPORTED: return "unsupported shape (head_dim must be 64, 72, 96, 104 or 128; d_model and d_ff multiples of 8)";
        case KRAKEN_ECAPACITY: return "capacity exceeded (batch, sequence length or buffer size)";
        case KRAKEN_ESTATE: return "call order violated (prefill first; decode batch must equal the prefill batch)";
        case KRAKEN_ECUDA: return "a CUDA call failed";
        default: return "unknown status";
    }
}

// ------------------------------------------------------------------ single steps

int kraken_op_embed(const int32_t *d_ids, int32_t n_tokens, int32_t seqlen, int32_t pos0, const void *wte,
                    const void *wpe, int32_t d_model, int32_t vocab, float *d_out, uint32_t *d_status, void *stream) {
    return launch_embed(d_ids, n_tokens, seqlen, pos0, (const uint16_t *)wte, (const uint16_t *)wpe, d_model, vocab,
                        d_out, d_status, static_cast<cudaStream_t>(stream));
}

int kraken_op_layernorm(const float *d_a, int64_t a_gstride, const float *d_y, const void *gamma, const void *beta,
                        int32_t groups, int32_t rows, int32_t d_model, float eps, void *d_out_bf16,
                        uint32_t *d_status, void *stream) {
    return launch_layernorm(d_a, a_gstride, d_y, (const uint16_t *)gamma, (const uint16_t *)beta, groups, rows,
                            d_model, eps, (uint16_t *)d_out_bf16, static_cast<cudaStream_t>(stream), nullptr, 0, 0,
                            d_status);
}

namespace {
int op_grouped_gemm(const kraken_gemm_args *g, const kraken_gemm_ln_args *ln, uint32_t *d_status, void *stream);
size_t ln_cnt_region(int groups, int m) { return align_up(gemm_ln_cnt_bytes(groups, m)); }
int ln_tile_of(const kraken_gemm_args *g) {
    return g->n_tile ? g->n_tile : gemm_pick_bn(GemmShape{g->groups, g->m, g->n_out, g->k});
}
}  // namespace

int kraken_op_grouped_gemm(const kraken_gemm_args *g, uint32_t *d_status, void *stream) {
    return op_grouped_gemm(g, nullptr, d_status, stream);
}

int kraken_gemm_ln_scratch_bytes(int32_t groups, int32_t m, int32_t n_out, int32_t k, int32_t n_tile, size_t *bytes) {
    if (!bytes || groups < 1 || m < 1 || n_out < 1 || k < 1) return KRAKEN_EINVAL;
    if (n_tile == 8 || (n_tile && n_tile != GEMM_TILE_PAIR && (n_tile < 32 || n_tile > 256 || n_tile % 32)))
        return KRAKEN_EUNSUPPORTED;
    const int bn = n_tile ? n_tile : gemm_pick_bn(GemmShape{groups, m, n_out, k});
    *bytes = ln_cnt_region(groups, m) + gemm_ln_parts_bytes(groups, m, n_out, bn);
    return KRAKEN_OK;
}

int kraken_op_grouped_gemm_ln(const kraken_gemm_args *g, const kraken_gemm_ln_args *ln, uint32_t *d_status,
                              void *stream) {
    if (!ln) return KRAKEN_EINVAL;
    return op_grouped_gemm(g, ln, d_status, stream);
}

namespace {
int op_grouped_gemm(const kraken_gemm_args *g, const kraken_gemm_ln_args *ln, uint32_t *d_status, void *stream) {
    if (!g || !g->a || !g->w) return KRAKEN_EINVAL;
    if (g->epilogue < KRAKEN_EPI_F32 || g->epilogue > KRAKEN_EPI_QKV) return KRAKEN_EINVAL;
    const int k = g->epilogue;
    const bool need_f32 = k == KRAKEN_EPI_F32 || k == KRAKEN_EPI_RESID_F32 || k == KRAKEN_EPI_RESID_SUM;
    const bool need_bf16 = k == KRAKEN_EPI_BF16 || k == KRAKEN_EPI_GELU_BF16 || k == KRAKEN_EPI_QKV;
    if ((need_f32 && !g->out_f32) || (need_bf16 && !g->out_bf16)) return KRAKEN_EINVAL;
    if ((k == KRAKEN_EPI_RESID_F32 || k == KRAKEN_EPI_RESID_SUM) && !g->resid) return KRAKEN_EINVAL;
    if (k == KRAKEN_EPI_RESID_SUM && !g->sum) return KRAKEN_EINVAL;
    if (k == KRAKEN_EPI_QKV) {
        if (!g->k_cache || !g->v_cache || g->seqlen < 1 || g->n_head < 1 || g->pos0 < 0) return KRAKEN_EINVAL;
        // q | k | v and head boundaries fall on 16-byte pieces; the q rows and cache rows must be 16-byte aligned
        if (g->n_kv_head < 0 || (g->n_kv_head > 0 && g->n_head % g->n_kv_head != 0)) return KRAKEN_EINVAL;
        const int n_kv = g->n_kv_head > 0 ? g->n_kv_head : g->n_head;
        if (g->head_dim % 8 != 0 || g->n_out != (g->n_head + 2 * n_kv) * g->head_dim || g->ld_out_bf16 % 8 != 0 ||
            g->out_bf16_gstride % 8 != 0 || g->cache_gstride % 8 != 0)
            return KRAKEN_EUNSUPPORTED;
    }
    GemmOperands op{g->a, g->a_gstride, g->lda, g->w, g->w_gstride, g->ldw, g->w_constant != 0};
    GemmShape s{g->groups, g->m, g->n_out, g->k};
    EpiParams e = epi_zero();
    e.kind = k;
    e.bias = (const uint16_t *)g->bias; e.bias_gstride = g->bias_gstride;
    e.out_f32 = g->out_f32; e.out_f32_gstride = g->out_f32_gstride; e.ld_out_f32 = g->ld_out_f32;
    e.out_bf16 = (uint16_t *)g->out_bf16; e.out_bf16_gstride = g->out_bf16_gstride; e.ld_out_bf16 = g->ld_out_bf16;
    e.resid = g->resid; e.resid_gstride = g->resid_gstride; e.ld_resid = g->ld_resid;
    e.sum = g->sum; e.ld_sum = g->ld_sum;
    e.k_cache = (uint16_t *)g->k_cache; e.v_cache = (uint16_t *)g->v_cache; e.cache_gstride = g->cache_gstride;
    e.seqlen = g->seqlen; e.pos0 = g->pos0; e.n_head = g->n_head; e.head_dim = g->head_dim; e.max_pos = g->max_pos;
    e.d_model = g->n_head * g->head_dim;
    e.n_kv_head = g->n_kv_head > 0 ? g->n_kv_head : g->n_head;
    e.gelu_tanh = g->gelu_tanh;
    int n_tile = g->n_tile;
    if (ln) {
        if (k != KRAKEN_EPI_RESID_F32 && k != KRAKEN_EPI_RESID_SUM) return KRAKEN_EINVAL;
        if (!ln->ln_out || !ln->gamma || !ln->d_scratch || !(ln->eps > 0.f)) return KRAKEN_EINVAL;
        if (n_tile == 8) return KRAKEN_EUNSUPPORTED;
        n_tile = ln_tile_of(g);
        const size_t cnt_bytes = ln_cnt_region(g->groups, g->m);
        if (ln->scratch_bytes < cnt_bytes + gemm_ln_parts_bytes(g->groups, g->m, g->n_out, n_tile)) return KRAKEN_ECAPACITY;
        e.ln_out = (uint16_t *)ln->ln_out; e.ln_out_gstride = ln->ln_out_gstride; e.ln_ld_out = ln->ld_ln_out;
        e.ln_gamma = (const uint16_t *)ln->gamma; e.ln_beta = (const uint16_t *)ln->beta; e.ln_gb_gstride = ln->gb_gstride;
        e.ln_y = ln->y; e.ln_ld_y = ln->ld_y;
        e.ln_eps = ln->eps;
        e.ln_cnt = reinterpret_cast<uint32_t *>(ln->d_scratch);
        e.ln_parts = reinterpret_cast<float4 *>(static_cast<uint8_t *>(ln->d_scratch) + cnt_bytes);
    }
    if (n_tile == 8) return launch_gemm_skinny(op, s, e, static_cast<cudaStream_t>(stream));
    return launch_gemm_tc(op, s, e, nullptr, nullptr, 0, n_tile, d_status, static_cast<cudaStream_t>(stream));
}
}  // namespace

int kraken_op_attention(const void *q, int64_t q_gstride, const void *k_cache, const void *v_cache,
                        int64_t cache_gstride, int64_t cache_bstride, int32_t groups, int32_t batch, int32_t seqlen,
                        int32_t pos0, int32_t n_head, int32_t n_kv_head, int32_t head_dim, int32_t max_pos,
                        void *out, int64_t out_gstride, void *stream) {
    if (n_head < 1 || n_kv_head < 0 || (n_kv_head > 0 && n_head % n_kv_head != 0)) return KRAKEN_EINVAL;
    AttnParams p;
    p.n_kv_head = n_kv_head;
    p.q = (const uint16_t *)q; p.q_gstride = q_gstride;
    p.k_cache = (const uint16_t *)k_cache; p.v_cache = (const uint16_t *)v_cache;
    p.cache_gstride = cache_gstride; p.cache_bstride = cache_bstride;
    p.groups = groups; p.batch = batch; p.seqlen = seqlen; p.pos0 = pos0; p.n_head = n_head; p.head_dim = head_dim;
    p.max_pos = max_pos; p.out = (uint16_t *)out; p.out_gstride = out_gstride;
    // one kernel serves every supported layout; a cache with gaps between its rows or heads is refused
    return launch_attention_tc(p, nullptr, nullptr, nullptr, nullptr, static_cast<cudaStream_t>(stream));
}

int kraken_op_decode_attention(const void *q, int64_t q_gstride, const void *k_cache, const void *v_cache,
                               int64_t cache_gstride, int64_t cache_bstride, int32_t groups, int32_t batch,
                               int32_t n_keys, int32_t n_head, int32_t n_kv_head, int32_t head_dim, int32_t max_pos,
                               int32_t splits, void *d_partials, size_t partial_bytes, void *out,
                               int64_t out_gstride, void *stream) {
    if (groups < 1 || batch < 1 || n_head < 1 || n_keys < 1) return KRAKEN_EINVAL;
    if (n_kv_head < 0 || (n_kv_head > 0 && n_head % n_kv_head != 0)) return KRAKEN_EINVAL;
    if (!decode_head_dim_ok(head_dim)) return KRAKEN_EUNSUPPORTED;
    if (splits == 0) splits = decode_attention_splits(groups, batch, n_head, n_keys);
    if (splits < 1 || splits > DECODE_MAX_SPLITS) return KRAKEN_EINVAL;
    if (splits > 1 && (!d_partials || partial_bytes < decode_attention_partial_bytes(groups, batch, n_head, head_dim, splits)))
        return KRAKEN_ECAPACITY;
    DecodeAttnParams p;
    p.q = (const uint16_t *)q; p.q_gstride = q_gstride;
    p.k_cache = (const uint16_t *)k_cache; p.v_cache = (const uint16_t *)v_cache;
    p.cache_gstride = cache_gstride; p.cache_bstride = cache_bstride;
    p.groups = groups; p.batch = batch; p.n_keys = n_keys; p.n_head = n_head; p.head_dim = head_dim;
    p.max_pos = max_pos; p.pos_dev = nullptr; p.splits = splits; p.partials = (float *)d_partials;
    p.out = (uint16_t *)out; p.out_gstride = out_gstride;
    p.n_kv_head = n_kv_head;
    return launch_attention_decode(p, static_cast<cudaStream_t>(stream));
}

int kraken_decode_attention_sizes(int32_t groups, int32_t batch, int32_t n_keys, int32_t n_head, int32_t head_dim,
                                  int32_t *splits, size_t *partial_bytes) {
    if (groups < 1 || batch < 1 || n_head < 1 || n_keys < 1 || !splits || !partial_bytes) return KRAKEN_EINVAL;
    if (!decode_head_dim_ok(head_dim)) return KRAKEN_EUNSUPPORTED;
    if (*splits == 0) *splits = decode_attention_splits(groups, batch, n_head, n_keys);
    if (*splits < 1 || *splits > DECODE_MAX_SPLITS) return KRAKEN_EINVAL;
    *partial_bytes = *splits > 1 ? decode_attention_partial_bytes(groups, batch, n_head, head_dim, *splits) : 0;
    return KRAKEN_OK;
}

}  // extern "C"
