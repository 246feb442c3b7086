#!/usr/bin/env python
"""Benchmark of the single-GPU Kraken prefill path (and of the CPU oracle as the reference arm).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C3] [--impl ours|reference]

One step = one whole prefill (embedding, L layers of N branches, W_concat, final LayerNorm,
unembedding of the last positions) over one batch of seeded synthetic tokens.  Rank 0 prints ONE
JSON line.  With N > 1 (torchrun) every rank runs an independent replica on its own GPU
("replicas only": the path has no inter-GPU step), timed between barriers, max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of ONE launch of the dominant kernel, from
# the ncu captures summarised under profiles/ (layer-shaped launches of paper_2408_07802_b200.cases).
NCU_TRAFFIC = {
    "C3": {"bytes": 855.9e6, "launch": "FFN up-projection (4 x 8192 x 8192 x 2048)", "algorithmic_bytes": 805.3e6,
           "source": "profiles/gemm_tc_pair_kernel_C3_gemm_up.md"},
    "C4": {"bytes": 541.3e6, "launch": "decode attention of one layer (1024 streams x 2048 keys)",
           "algorithmic_bytes": 537.1e6, "source": "profiles/attn_decode_kernel_C4.md"},
}

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
PAPER_CONTEXT = ("paper: 35.6% geomean TTFT speedup of Kraken over standard Transformers, TensorRT-LLM fp16 on "
                 "8xA100-40GB NVSwitch (another machine and other shapes: context, not a target)")


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples of one GPU while a region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if not self.proc:
            return out
        self.proc.terminate()
        try:
            text, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            text = ""
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in text.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def host_weight_bits(w):
    import kraken_inputs as ki
    return {k: (None if v is None else ki.bf16_tensor_to_bits(v)) for k, v in w.items()}


HALF = False   # set from --dtype: the oracle then reads the weight patterns as IEEE half


def oracle_tokens_per_s(shape, wb, ids, n_tokens):
    """Oracle prefill of the first n_tokens of one sequence (last-position logits only)."""
    import oracle
    orc = oracle.Oracle(shape, wb, half=HALF)
    t0 = time.perf_counter()
    orc.prefill(ids[:n_tokens], logits_from=n_tokens - 1)
    dt = time.perf_counter() - t0
    orc.close()
    return n_tokens / dt, dt


def run_reference(args, shape):
    """Reference arm: the CPU oracle, as it stands, on a bounded sample of the same workload."""
    import torch
    import kraken_inputs as ki
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    w = ki.make_weights(shape, seed=0, device=dev, dtype=args.dtype)
    wb = host_weight_bits(w)
    del w
    ids = ki.uniform_tokens(1, shape.vocab, shape.batch, shape.seqlen)[0].numpy()
    n = max(1, min(shape.seqlen, args.ref_tokens))
    for _ in range(args.warmup):
        oracle_tokens_per_s(shape, wb, ids, n)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_tokens_per_s(shape, wb, ids, n)
    dt = (time.perf_counter() - t0) / args.steps
    value = n / dt
    sample = f"oracle prefill of the first {n} tokens of sequence 0 of {shape.name} per step"
    line = {
        "impl": "reference", "metric": "prefill_tokens_per_s", "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32 values, f64 accumulation",
        "data": "synthetic", "config": workload_config(shape, args),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(shape, args):
    what = "decode after prefill" if shape.decode_steps else "prefill"
    cfg = {"workload": f"{shape.name} {what}", "n_branch": shape.n_branch, "n_layer": shape.n_layer,
           "d_model": shape.d_model, "n_head": shape.n_head, "n_kv_head": shape.kv_heads, "d_ff": shape.d_ff,
           "vocab": shape.vocab,
           "batch": shape.batch, "seqlen": shape.seqlen, "tokens_per_step": shape.batch * shape.seqlen,
           "parallelism": f"replicas x{args.gpus}" if args.gpus > 1 else "single GPU",
           "l2": "inputs larger than L2 (weights read every step exceed 126 MB)"
                 if weight_bytes(shape) > 126e6 else "L2 flushed between steps",
           "context": PAPER_CONTEXT}
    if not shape.decode_steps and shape.batch * shape.seqlen > 32:
        cfg["last_layer"] = ("past its qkv GEMM the last layer runs for the last position of every sequence only (the "
                             "logits of the other positions are not part of the call); that work is not in the FLOP counts")
    paper_ms = paper_ttft_ms(shape)
    if paper_ms is not None:
        cfg["paper_ttft_ms"] = paper_ms
        cfg["paper_setup"] = (f"Tables 4/5: this engine shape, fp16, batch 1, one branch per GPU on "
                              f"{shape.n_branch} x A100-40GB (another machine and precision: context, not a target)")
    return cfg


def paper_ttft_ms(shape):
    """The TTFT the paper prints for this engine shape and context (Tables 4 and 5), else None."""
    import kraken_inputs as ki
    if shape.batch != 1 or shape.decode_steps:
        return None
    return ki.PAPER_TTFT_MS.get(shape.name, {}).get(shape.seqlen)


def weight_bytes(s):
    return 2 * (s.n_layer * s.n_branch * (s.d_model * s.qkv_width + s.d_model ** 2 + 2 * s.d_model * s.d_ff)
                + s.vocab * s.d_model)


def decode_bytes(shape, t):
    """Bytes one decode step must move at cache length t: every weight once, K and V rows 0..t."""
    s = shape
    w = 2 * (s.n_layer * s.n_branch * (s.d_model * s.qkv_width + s.d_model ** 2 + 2 * s.d_model * s.d_ff)
             + s.vocab * s.d_model + s.n_branch * s.d_model ** 2)
    kv = 2 * s.n_layer * s.n_branch * s.batch * (t + 1) * s.kv_heads * s.head_dim * 2
    return w, kv


def run_decode(args, shape, kr, ki, replicas, torch):
    """C4: prefill `seqlen` tokens per sequence, then time greedy decode steps (one step = one
    kraken_decode_step over the whole batch; the arg-max feeding the next step is the caller's)."""
    rank, local_rank, world = replicas.rank_env()
    dev = f"cuda:{local_rank}"
    steps = min(args.steps, shape.decode_steps)
    w = ki.make_weights(shape, seed=0, device=dev, dtype=args.dtype)
    model = kr.KrakenModel(kr.make_config(shape), w, dev, dtype=args.dtype)
    tok = ki.uniform_tokens(replicas.token_seed(rank), shape.vocab, shape.batch, shape.seqlen, dev)
    logits = torch.empty(shape.batch, shape.vocab, dtype=torch.float32, device=dev)

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    def start():
        model.prefill(tok, logits)
        return logits.argmax(1).to(torch.int32)

    nxt = start()
    for _ in range(max(args.warmup, 3)):
        model.decode_step(nxt, logits)
        nxt = logits.argmax(1).to(torch.int32)
    nxt = start()
    barrier()
    model.profile_read()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.25)
    e0 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    e1 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    barrier()
    for i in range(steps):
        e0[i].record()
        model.decode_step(nxt, logits)
        e1[i].record()
        nxt = logits.argmax(1).to(torch.int32)
    barrier()
    clocks = sampler.stop()
    per_step = [a.elapsed_time(b) for a, b in zip(e0, e1)]
    _, launches = model.profile_read()
    ms_per_step = replicas.max_over_ranks(sum(per_step), dev) / steps
    value = replicas.whole_job_throughput(shape.batch, ms_per_step, world)

    # per-kernel device time: the same steps again from the same start, events around every launch
    nxt = start()
    model.profile_read()
    model.profile_enable(True)
    for _ in range(steps):
        model.decode_step(nxt, logits)
        nxt = logits.argmax(1).to(torch.int32)
    prof_ms, prof_n = model.profile_read()
    model.profile_enable(False)

    # end to end: host token ids in, host logits out, every step
    nxt = start()
    h_tok = nxt.cpu().pin_memory()
    h_log = torch.empty(shape.batch, shape.vocab, dtype=torch.float32).pin_memory()
    barrier()
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record()
    for _ in range(steps):
        model.decode_step_host(h_tok, h_log)
        h_tok.copy_(h_log.argmax(1).to(torch.int32))
    s1.record()
    barrier()
    e2e_ms = replicas.max_over_ranks(s0.elapsed_time(s1), dev) / steps
    status = model.device_status()
    if rank != 0:
        return

    peaks, peak_kind = load_peaks()
    t_mid = shape.seqlen + steps // 2
    wb_, kvb = decode_bytes(shape, t_mid)
    total_bytes = wb_ + kvb
    attn_ms = prof_ms["attention"] / steps
    attn_launch = prof_n["attention"] / steps
    kv_per_layer = kvb / shape.n_layer
    attn_gbs = kvb / (attn_ms * 1e-3) / 1e9 if attn_ms > 0 else 0.0
    kernels = {k: {"ms_per_step": v / steps, "launches_per_step": prof_n[k] / steps} for k, v in prof_ms.items()}
    gemm_ms = sum(prof_ms[k] for k in ("gemm_qkv", "gemm_proj", "gemm_up", "gemm_down", "tail")) / steps
    line = {
        "metric": "decode_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": args.dtype, "data": "synthetic", "config": workload_config(shape, args),
        "hbm_gbs": total_bytes / (ms_per_step * 1e-3) / 1e9,
        "frac_of_measured_hbm": total_bytes / (ms_per_step * 1e-3) / 1e9 / peaks["hbm_gbs"],
        "bytes_per_step": {"weights": wb_, "kv_cache": kvb, "at_cache_length": t_mid},
        "clocks": clocks,
        "e2e": {"value": replicas.whole_job_throughput(shape.batch, e2e_ms, world), "unit": "tokens/s",
                "ms_per_step": e2e_ms, "h2d_bytes_per_step": shape.batch * 4,
                "d2h_bytes_per_step": shape.batch * shape.vocab * 4},
        "gpu_launches": int(sum(launches.values())),
        "roofline": {"bound": "hbm", "kernel": "attn_decode_kernel (split-KV cache streaming)",
                     "achieved": attn_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": attn_gbs / peaks["hbm_gbs"], "peak_source": f"hbm_gbs of {peak_kind}",
                     "bytes_per_launch": kv_per_layer, "launches_per_step": attn_launch,
                     "avg_launch_ms": attn_ms / shape.n_layer,
                     "timed_in": "separate pass of the same steps with events around every launch",
                     "traffic": NCU_TRAFFIC.get(shape.name, {}).get("bytes"),
                     "traffic_note": NCU_TRAFFIC.get(shape.name)},
        "weight_streaming": {"ms_per_step": gemm_ms, "gbs": wb_ / (gemm_ms * 1e-3) / 1e9 if gemm_ms > 0 else 0.0},
        "kernels": kernels, "device_status": status,
    }
    if world == 1 and not args.no_cpu_baseline:
        import oracle
        hb = host_weight_bits(w)
        ctx, n_dec = 256, 8
        orc = oracle.Oracle(shape, hb, half=HALF)
        ids = tok[0].cpu().numpy()
        orc.prefill(ids[:ctx], logits_from=ctx - 1)
        t0 = time.perf_counter()
        nid = int(ids[ctx])
        for _ in range(n_dec):
            nid = int(orc.decode_step(nid).argmax())
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": n_dec / dt, "unit": "tokens/s", "cores": oracle.num_threads(),
                                "kind": "oracle", "sample": f"{n_dec} oracle decode steps of ONE sequence after a "
                                f"{ctx}-token prefill ({dt:.1f} s); the GPU figure is {shape.batch} sequences at "
                                f"context {shape.seqlen}"}
    print(json.dumps(line))


def prefill_leg(name, args, kr, ki, torch, dev, local_rank, steps=20):
    """A short prefill measurement of another BASELINE config, for the `other_configs` key of the default line:
    same protocol as the headline (warm-up, events on the launching stream, L2 flushed between steps when the
    weights fit in it, clock samples during the timed steps, a second pass with events around every launch)."""
    shape = ki.CONFIGS[name]
    w = ki.make_weights(shape, seed=0, device=dev, dtype=args.dtype)
    model = kr.KrakenModel(kr.make_config(shape), w, dev, dtype=args.dtype)
    tok = ki.uniform_tokens(1, shape.vocab, shape.batch, shape.seqlen, dev)
    logits = torch.empty(shape.batch, shape.vocab, dtype=torch.float32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if weight_bytes(shape) <= 126e6 else None
    for _ in range(5):
        model.prefill(tok, logits)
    torch.cuda.synchronize()
    model.profile_read()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.25)
    e0 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    e1 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    for i in range(steps):
        if flush is not None:
            flush.zero_()
        e0[i].record()
        model.prefill(tok, logits)
        e1[i].record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    per_step = sorted(a.elapsed_time(b) for a, b in zip(e0, e1))
    _, launches = model.profile_read()
    ms = sum(per_step) / steps
    model.profile_enable(True)
    for _ in range(steps):
        if flush is not None:
            flush.zero_()
        model.prefill(tok, logits)
    prof_ms, prof_n = model.profile_read()
    model.profile_enable(False)
    status = model.device_status()
    model.close()
    peaks, _ = load_peaks()
    fl = ki.algorithmic_flops(shape, last_positions_only=shape.batch * shape.seqlen > 32)
    tokens = shape.batch * shape.seqlen
    return {
        "workload": f"{name} prefill", "batch": shape.batch, "seqlen": shape.seqlen, "steps": steps,
        "ttft_ms": ms, "ttft_ms_median": per_step[len(per_step) // 2], "ttft_ms_min": per_step[0],
        "tokens_per_s": tokens / (ms * 1e-3),
        "model_tflops": fl["total"] / (ms * 1e-3) / 1e12,
        "frac_of_nominal_2250": fl["total"] / (ms * 1e-3) / 2.25e15,
        "frac_of_measured_sustained": fl["total"] / (ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
        "gpu_launches_per_step": int(sum(launches.values())) // steps,
        "l2": "flushed between steps" if flush is not None else "weights exceed L2",
        "kernels_ms_per_step": {k: v / steps for k, v in prof_ms.items()},
        "clocks": clocks, "device_status": status,
    }


def decode_leg(name, args, kr, ki, torch, dev, local_rank):
    """The decode config for the `other_configs` key: prefill once, then all of the config's greedy decode steps
    (events around every step), then the same steps with events around every launch (single chain)."""
    shape = ki.CONFIGS[name]
    steps = shape.decode_steps
    w = ki.make_weights(shape, seed=0, device=dev, dtype=args.dtype)
    model = kr.KrakenModel(kr.make_config(shape), w, dev, dtype=args.dtype)
    tok = ki.uniform_tokens(1, shape.vocab, shape.batch, shape.seqlen, dev)
    logits = torch.empty(shape.batch, shape.vocab, dtype=torch.float32, device=dev)

    def start():
        model.prefill(tok, logits)
        return logits.argmax(1).to(torch.int32)

    nxt = start()
    for _ in range(3):
        model.decode_step(nxt, logits)
        nxt = logits.argmax(1).to(torch.int32)
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record()
    nxt = start()
    p1.record()
    torch.cuda.synchronize()
    prefill_ms = p0.elapsed_time(p1)
    model.profile_read()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.25)
    e0 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    e1 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    for i in range(steps):
        e0[i].record()
        model.decode_step(nxt, logits)
        e1[i].record()
        nxt = logits.argmax(1).to(torch.int32)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = sum(a.elapsed_time(b) for a, b in zip(e0, e1)) / steps
    _, launches = model.profile_read()
    nxt = start()
    model.profile_read()
    model.profile_enable(True)
    for _ in range(steps):
        model.decode_step(nxt, logits)
        nxt = logits.argmax(1).to(torch.int32)
    prof_ms, prof_n = model.profile_read()
    model.profile_enable(False)
    status = model.device_status()
    model.close()
    peaks, _ = load_peaks()
    wb_, kvb = decode_bytes(shape, shape.seqlen + steps // 2)
    gbs = (wb_ + kvb) / (ms * 1e-3) / 1e9
    attn_ms = prof_ms["attention"] / steps
    gemm_ms = sum(prof_ms[k] for k in ("gemm_qkv", "gemm_proj", "gemm_up", "gemm_down", "tail")) / steps
    return {
        "workload": f"{name} decode after prefill", "batch": shape.batch, "context": shape.seqlen, "steps": steps,
        "prefill_ms": prefill_ms, "ms_per_step": ms, "tokens_per_s": shape.batch / (ms * 1e-3),
        "hbm_gbs": gbs, "frac_of_measured_hbm": gbs / peaks["hbm_gbs"], "frac_of_nominal_8000": gbs / 8000.0,
        "bytes_per_step": {"weights": wb_, "kv_cache": kvb},
        "attention_gbs_single_chain": kvb / (attn_ms * 1e-3) / 1e9 if attn_ms > 0 else None,
        "weight_streaming_gbs_single_chain": wb_ / (gemm_ms * 1e-3) / 1e9 if gemm_ms > 0 else None,
        "gpu_launches_per_step": int(sum(launches.values())) // steps,
        "kernels_ms_per_step_single_chain": {k: v / steps for k, v in prof_ms.items()},
        "clocks": clocks, "device_status": status,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="C3")
    ap.add_argument("--seqlen", type=int, default=0,
                    help="prompt length override (the paper's engine shapes K* were timed at 128 and 2048)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f16"],
                    help="16-bit storage type: bf16 (libkraken.so) or IEEE half (libkraken_f16.so, the paper's precision)")
    ap.add_argument("--ref-tokens", type=int, default=8, help="tokens per step of the reference arm")
    ap.add_argument("--cpu-baseline-seconds", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layernorm", default="auto", choices=["auto", "fused", "fused-down"],
                    help="fused: every LayerNorm inside the GEMM kernel that finishes its rows; fused-down: only behind "
                         "the FFN down-projection (for comparison with the default, separate LayerNorm launches)")
    ap.add_argument("--headline-only", action="store_true",
                    help="skip the short legs of the other BASELINE configs that the default C3 run appends")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    import kraken_inputs as ki
    global HALF
    HALF = args.dtype == "f16"
    shape = ki.CONFIGS[args.workload]
    if args.seqlen:
        import dataclasses
        shape = dataclasses.replace(shape, seqlen=args.seqlen)
    if args.impl == "reference":
        run_reference(args, shape)
        return

    import torch
    import paper_2408_07802_b200 as kr
    from paper_2408_07802_b200 import build as kbuild

    from paper_2408_07802_b200 import replicas
    rank, local_rank, world = replicas.rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if args.layernorm != "auto":
        with kr.storage_dtype(args.dtype):
            kr.set_tuning(kr.TUNE_LN_FUSION, 2 if args.layernorm == "fused" else 3)
    dist = None
    if world > 1:
        dist = replicas.init_process_group("nccl", torch.device(dev))
    if rank == 0:
        kbuild.build(dtype=args.dtype)
    if dist:
        dist.barrier()
    kr.lib(args.dtype)
    if shape.decode_steps:
        if args.steps == 10:
            args.steps = shape.decode_steps
        run_decode(args, shape, kr, ki, replicas, torch)
        if dist:
            dist.destroy_process_group()
        return

    w = ki.make_weights(shape, seed=0, device=dev, dtype=args.dtype)
    model = kr.KrakenModel(kr.make_config(shape), w, dev, dtype=args.dtype)
    tok = ki.uniform_tokens(replicas.token_seed(rank), shape.vocab, shape.batch, shape.seqlen, dev)
    logits = torch.empty(shape.batch, shape.vocab, dtype=torch.float32, device=dev)
    flush = None
    if weight_bytes(shape) <= 126e6:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def step():
        if flush is not None:
            flush.zero_()
        model.prefill(tok, logits)

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    model.profile_read()  # reset the launch counters

    # ---- timed region: K steps, device time by events on the launching stream
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.25)
    e0 = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    e1 = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    barrier()
    for i in range(args.steps):
        if flush is not None:
            flush.zero_()
        e0[i].record()
        model.prefill(tok, logits)
        e1[i].record()
    barrier()
    clocks = sampler.stop()
    per_step = [a.elapsed_time(b) for a, b in zip(e0, e1)]
    total_ms = sum(per_step)
    _, launches = model.profile_read()
    gpu_launches = int(sum(launches.values()))
    total_ms = replicas.max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / args.steps
    tokens = shape.batch * shape.seqlen
    value = replicas.whole_job_throughput(tokens, ms_per_step, world)

    # ---- end to end through the host-buffer call: pinned tokens in, logits out, every step
    h_tok = tok.cpu().pin_memory()
    h_log = torch.empty(shape.batch, shape.vocab, dtype=torch.float32).pin_memory()
    for _ in range(2):
        model.prefill_host(h_tok, h_log)
    barrier()
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record()
    for _ in range(args.steps):
        if flush is not None:
            flush.zero_()
        model.prefill_host(h_tok, h_log)
    s1.record()
    barrier()
    e2e_ms = s0.elapsed_time(s1) / args.steps
    e2e_ms = replicas.max_over_ranks(e2e_ms, dev)
    e2e_value = replicas.whole_job_throughput(tokens, e2e_ms, world)
    # ---- the same K steps again with every launch bracketed by events: per-kernel device time
    model.profile_read()            # (drops the counts of the end-to-end steps)
    model.profile_enable(True)
    for _ in range(args.steps):
        step()
    prof_ms, prof_n = model.profile_read()
    model.profile_enable(False)

    status = model.device_status()

    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    peaks, peak_kind = load_peaks()
    # the call returns last-position logits, so the last layer runs on one row per sequence past its qkv GEMM: the
    # work that is thereby not needed is not counted (kraken_inputs.algorithmic_flops)
    short_last = tokens > 32
    fl = ki.algorithmic_flops(shape, last_positions_only=short_last)
    gemm_ms = sum(prof_ms[k] for k in ("gemm_qkv", "gemm_proj", "gemm_up", "gemm_down")) / args.steps
    gemm_launches = sum(prof_n[k] for k in ("gemm_qkv", "gemm_proj", "gemm_up", "gemm_down")) // args.steps
    achieved = fl["gemm"] / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
    peak = peaks["bf16_tflops_sustained"]
    T, N, L, d, F = tokens, shape.n_branch, shape.n_layer, shape.d_model, shape.d_ff
    rows_rest = T * (L - 1) + shape.batch if short_last else T * L      # token rows past the qkv GEMMs, over all layers
    kind_flops = {"gemm_qkv": 2.0 * T * N * L * 3 * d * d, "gemm_proj": 2.0 * rows_rest * N * d * d,
                  "gemm_up": 2.0 * rows_rest * N * d * F, "gemm_down": 2.0 * rows_rest * N * d * F,
                  "attention": fl["attn"]}
    kernels = {}
    for k, ms in prof_ms.items():
        ent = {"ms_per_step": ms / args.steps, "launches_per_step": prof_n[k] // args.steps}
        if k in kind_flops and ms > 0:
            ent["tflops"] = kind_flops[k] / (ms / args.steps * 1e-3) / 1e12
        kernels[k] = ent
    line = {
        "metric": "prefill_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "ttft_ms": ms_per_step,
        "higher_is_better": True, "scaling": "weak",
        # tokens/s against the paper's figure for the same engine shape and context, where it prints one
        "vs_baseline": (value / (shape.seqlen / (paper_ttft_ms(shape) * 1e-3))
                        if paper_ttft_ms(shape) is not None and world == 1 else None),
        "dtype": args.dtype,
        "data": "synthetic", "config": workload_config(shape, args),
        "model_tflops": fl["total"] / (ms_per_step * 1e-3) / 1e12,
        "frac_of_nominal_2250": fl["total"] / (ms_per_step * 1e-3) / 2.25e15,
        "frac_of_measured_sustained": fl["total"] / (ms_per_step * 1e-3) / 1e12 / peak,
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "tokens/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": tokens * 4, "d2h_bytes_per_step": shape.batch * shape.vocab * 4},
        "gpu_launches": gpu_launches,
        "roofline": {"bound": "tensor", "kernel": "gemm_tc_pair_kernel / gemm_tc_kernel (grouped tcgen05 GEMM: qkv, proj, up, down)",
                     "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                     "peak_source": f"bf16_tflops_sustained of {peak_kind}",
                     "launches_per_step": int(gemm_launches), "avg_launch_ms": gemm_ms / max(1, gemm_launches),
                     "flops_per_step": fl["gemm"], "timed_in": "separate pass of the same K steps with events "
                     "around every launch",
                     "traffic": NCU_TRAFFIC.get(shape.name, {}).get("bytes"),
                     "traffic_note": NCU_TRAFFIC.get(shape.name)},
        "kernels": kernels,
        "device_status": status,
    }
    if world == 1 and not args.no_cpu_baseline:
        import oracle
        wb = host_weight_bits(w)
        ids = tok[0].cpu().numpy()
        probe_n = min(shape.seqlen, 4)
        rate, _ = oracle_tokens_per_s(shape, wb, ids, probe_n)
        n = int(max(probe_n, min(shape.seqlen, rate * args.cpu_baseline_seconds)))
        rate, dt = oracle_tokens_per_s(shape, wb, ids, n)
        line["cpu_baseline"] = {"value": rate, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
                                "sample": f"oracle prefill of the first {n} tokens of sequence 0 ({dt:.1f} s)"}
    if world == 1 and args.workload == "C3" and not args.seqlen and not args.headline_only:
        # the other four BASELINE configs, measured in the same run (each leg builds and frees its own model)
        model.close()
        del model, w, tok, logits
        torch.cuda.empty_cache()
        others = {}
        for name in ("C0", "C1", "C2"):
            others[name] = prefill_leg(name, args, kr, ki, torch, dev, local_rank)
            torch.cuda.empty_cache()
        others["C4"] = decode_leg("C4", args, kr, ki, torch, dev, local_rank)
        line["other_configs"] = others
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
