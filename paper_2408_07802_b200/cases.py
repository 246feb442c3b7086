"""Single-kernel cases at the layer shapes of a workload, through the C ABI's step entry points.

    python -m paper_2408_07802_b200.cases gemm_up --workload C3 --reps 5

Each case builds one layer's worth of seeded inputs (a few hundred MB, larger than L2), runs the
kernel `--warmup` + `--reps` times and prints the CUDA-event time per launch with the achieved
TFLOP/s or GB/s.  It is the command the ncu captures under profiles/ were taken with.
"""
from __future__ import annotations

import argparse
import json

import torch

import kraken_inputs as ki
import paper_2408_07802_b200 as kr

DEV = "cuda:0"


def _gemm_args(kind, s, batch, seqlen, n_tile=0):
    N, d, F, H = s.n_branch, s.d_model, s.d_ff, s.n_head
    hd = d // H
    T = batch * seqlen
    plain = kind.endswith("_plain")       # same shape, cheapest epilogue (bf16 store): isolates the mainloop
    kind = kind.replace("_plain", "")
    resid_only = kind == "gemm_down_resid"   # the down-projection without the cross-branch sum (short prompts)
    kind = kind.replace("_resid", "")
    K, Nout = {"gemm_qkv": (d, 3 * d), "gemm_proj": (d, d), "gemm_up": (d, F), "gemm_down": (F, d)}[kind]
    a = ki.normal_bf16(11, 0, (N, T, K), 1.0, DEV)
    w = ki.normal_bf16(11, 1, (N, Nout, K), 0.02, DEV)
    bias = ki.normal_bf16(11, 2, (N, Nout), 0.02, DEV)
    g = kr.GemmArgs()
    g.a, g.a_gstride, g.lda = a.data_ptr(), T * K, K
    g.w, g.w_gstride, g.ldw = w.data_ptr(), Nout * K, K
    g.bias, g.bias_gstride = bias.data_ptr(), Nout
    g.groups, g.m, g.n_out, g.k, g.n_tile = N, T, Nout, K, n_tile
    keep = [a, w, bias]
    out_bytes = 0
    if plain:
        o = torch.empty(N, T, Nout, dtype=torch.bfloat16, device=DEV)
        g.epilogue = kr.EPI_BF16
        g.out_bf16, g.out_bf16_gstride, g.ld_out_bf16 = o.data_ptr(), T * Nout, Nout
        keep += [o]
        out_bytes = N * T * Nout * 2
    elif kind == "gemm_qkv":
        q = torch.empty(N, T, d, dtype=torch.bfloat16, device=DEV)
        cache = torch.empty(N, 2, batch, H, seqlen, hd, dtype=torch.bfloat16, device=DEV)
        g.epilogue = kr.EPI_QKV
        g.out_bf16, g.out_bf16_gstride, g.ld_out_bf16 = q.data_ptr(), T * d, d
        g.k_cache, g.v_cache, g.cache_gstride = cache[0, 0].data_ptr(), cache[0, 1].data_ptr(), cache.stride(0)
        g.seqlen, g.pos0, g.n_head, g.head_dim, g.max_pos = seqlen, 0, H, hd, seqlen
        keep += [q, cache]
        out_bytes = N * T * 3 * d * 2
    elif kind == "gemm_up":
        o = torch.empty(N, T, F, dtype=torch.bfloat16, device=DEV)
        g.epilogue = kr.EPI_GELU_BF16
        g.out_bf16, g.out_bf16_gstride, g.ld_out_bf16 = o.data_ptr(), T * F, F
        keep += [o]
        out_bytes = N * T * F * 2
    else:
        o = torch.empty(N, T, d, dtype=torch.float32, device=DEV)
        r = torch.zeros(N, T, d, dtype=torch.float32, device=DEV)
        g.out_f32, g.out_f32_gstride, g.ld_out_f32 = o.data_ptr(), T * d, d
        g.resid, g.resid_gstride, g.ld_resid = r.data_ptr(), T * d, d
        keep += [o, r]
        out_bytes = N * T * d * 8
        if kind == "gemm_down" and not resid_only:
            ssum = torch.empty(T, d, dtype=torch.float32, device=DEV)
            g.epilogue = kr.EPI_RESID_SUM
            g.sum, g.ld_sum = ssum.data_ptr(), d
            keep += [ssum]
            out_bytes += T * d * 4
        else:
            g.epilogue = kr.EPI_RESID_F32
    flops = 2.0 * N * T * K * Nout
    byts = N * (T * K + Nout * K) * 2 + out_bytes
    return g, keep, flops, byts


def run_case(kind: str, workload: str, reps: int, warmup: int, n_tile: int = 0, batch=None, seqlen=None,
             graph_launches: int = 0, kv_heads: int = 0):
    s = ki.CONFIGS[workload]
    batch = batch or s.batch
    seqlen = seqlen or s.seqlen
    N, d, H = s.n_branch, s.d_model, s.n_head
    hd = d // H
    T = batch * seqlen
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    if kind.startswith("decode_gemm_"):
        # the same projection with one row per sequence (decode step): weight streaming
        g, keep, flops, byts = _gemm_args(kind.replace("decode_", ""), s, batch, 1, 8)
        if g.epilogue == kr.EPI_RESID_SUM:
            g.epilogue = kr.EPI_RESID_F32
        fn = lambda: kr.op_grouped_gemm(g, status)
    elif kind.startswith("gemm_"):
        g, keep, flops, byts = _gemm_args(kind, s, batch, seqlen, n_tile)
        fn = lambda: kr.op_grouped_gemm(g, status)
    elif kind == "attention":
        q = ki.normal_bf16(12, 0, (N, T, d), 1.0, DEV)
        kc = ki.normal_bf16(12, 1, (N, batch, H, seqlen, hd), 1.0, DEV)
        vc = ki.normal_bf16(12, 2, (N, batch, H, seqlen, hd), 1.0, DEV)
        fn = lambda: kr.op_attention(q, kc, vc, batch, seqlen, 0, H)
        flops = float(N * batch * H) * 4 * hd * (seqlen * (seqlen + 1) / 2)
        byts = 4 * N * T * d * 2
    elif kind == "decode_attention":
        ctx = seqlen
        Hkv = kv_heads or s.kv_heads          # fewer key/value heads than heads: grouped-query attention
        q = ki.normal_bf16(12, 0, (N, batch, d), 1.0, DEV)
        kc = ki.normal_bf16(12, 1, (N, batch, Hkv, ctx, hd), 1.0, DEV)
        vc = ki.normal_bf16(12, 2, (N, batch, Hkv, ctx, hd), 1.0, DEV)
        sp, nb = kr.decode_attention_sizes(N, batch, ctx, H, hd, n_tile)
        part = torch.empty(max(nb, 16), dtype=torch.uint8, device=DEV)
        fn = lambda: kr.op_decode_attention(q, kc, vc, ctx, sp, part)
        flops = 4.0 * N * batch * ctx * d
        byts = 2 * N * batch * ctx * Hkv * hd * 2 + 2 * N * batch * d * 2
    elif kind == "layernorm":
        a = ki.normal_bf16(13, 0, (N, T, d), 1.0, DEV).float()
        y = ki.normal_bf16(13, 1, (T, d), 1.0, DEV).float()
        gamma = torch.ones(N, d, dtype=torch.bfloat16, device=DEV)
        beta = torch.zeros(N, d, dtype=torch.bfloat16, device=DEV)
        fn = lambda: kr.op_layernorm(a, y, gamma, beta, status=status)
        flops = 0.0
        byts = N * T * d * 4 + T * d * 4 + N * T * d * 2
    else:
        raise SystemExit(f"unknown case {kind}")
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    if graph_launches:
        # short kernels: replay `graph_launches` back-to-back launches from a CUDA graph, so that the host's
        # launch pace does not enter the measurement
        cg = torch.cuda.CUDAGraph()
        with torch.cuda.graph(cg):
            for _ in range(graph_launches):
                fn()
        cg.replay()
        torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for e0, e1 in ev:
        e0.record()
        if graph_launches:
            cg.replay()
        else:
            fn()
        e1.record()
    torch.cuda.synchronize()
    ms = sorted(e0.elapsed_time(e1) / max(1, graph_launches) for e0, e1 in ev)
    med = ms[len(ms) // 2]
    out = {"case": kind, "workload": workload, "batch": batch, "seqlen": seqlen, "n_tile": n_tile,
           "ms_median": med, "ms_min": ms[0], "tflops": flops / (med * 1e-3) / 1e12,
           "gbs": byts / (med * 1e-3) / 1e9, "algorithmic_bytes": byts, "flops": flops,
           "status": int(status.item())}
    print(json.dumps(out))
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", help="gemm_qkv | gemm_proj | gemm_up | gemm_down | gemm_down_resid | attention | layernorm | decode_attention | decode_gemm_{qkv,proj,up,down} | all | decode_all")
    ap.add_argument("--workload", default="C3")
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=2)
    ap.add_argument("--n-tile", type=int, default=0, help="GEMM N tile, or split count for decode_attention")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--seqlen", type=int, default=None)
    ap.add_argument("--graph", type=int, default=0, help="time this many launches replayed from one CUDA graph")
    ap.add_argument("--kv-heads", type=int, default=0, help="key/value heads of decode_attention (default: the workload's)")
    a = ap.parse_args()
    kinds = [a.case]
    if a.case == "all":
        kinds = ["gemm_qkv", "gemm_proj", "gemm_up", "gemm_down", "attention", "layernorm"]
    elif a.case == "decode_all":
        kinds = ["decode_gemm_qkv", "decode_gemm_proj", "decode_gemm_up", "decode_gemm_down", "decode_attention"]
    for k in kinds:
        run_case(k, a.workload, a.reps, a.warmup, a.n_tile, a.batch, a.seqlen, a.graph, a.kv_heads)


if __name__ == "__main__":
    main()
