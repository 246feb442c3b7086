"""Branch-parallel prefill: the paper's own deployment (Fig. 3, App. A.2) - every device holds some of the N
branches of every layer and the cross-branch sum of Algorithm 1 is an all-reduce between devices that runs
while the next layer's attention half computes.

The arithmetic stays in the CUDA library (`kraken_stage_*`); this module only orders the pieces and the
collective.  It is written against two small interfaces so that the same ordering can be exercised without
GPUs: an *engine* (the stage calls of one rank) and a *group* (sum over ranks).

    engine.stage_begin(tokens); engine.stage_buffers() -> (x0, local_sum)
    engine.stage_attention(l); engine.stage_ffn(l, y); engine.stage_concat() -> z; engine.stage_head(z) -> logits
    group.all_reduce_start(tensor) -> handle;  group.wait(handle)

`slice_weights` cuts a full model's weights into the part one rank holds.
"""
from __future__ import annotations

from typing import Dict, List, Optional

import torch


def slice_weights(weights: Dict[str, Optional[torch.Tensor]], n_branch: int, first: int, count: int,
                  with_concat_bias: bool) -> Dict[str, Optional[torch.Tensor]]:
    """The weights of branches first .. first+count-1 of a model with n_branch branches: per-branch tensors
    ([L][N]...) are cut along the branch axis, W_concat ([d][N*d]) along its input columns; the embedding
    tables and the final LayerNorm are shared.  b_concat goes to exactly one rank (with_concat_bias)."""
    out: Dict[str, Optional[torch.Tensor]] = {}
    for k, t in weights.items():
        if t is None:
            out[k] = None
        elif k in ("wte", "wpe", "lnf_g", "lnf_b"):
            out[k] = t
        elif k == "w_concat":
            d = t.shape[0]
            out[k] = t.reshape(d, n_branch, d)[:, first:first + count].reshape(d, count * d).contiguous()
        elif k == "b_concat":
            out[k] = t if with_concat_bias else None
        else:
            out[k] = t[:, first:first + count].contiguous()
    return out


class TorchDistGroup:
    """Sum over the ranks of a torch.distributed process group.  With the NCCL backend the all-reduce is
    enqueued behind the work already on the current stream and runs on the backend's own stream, so whatever
    is enqueued on the current stream afterwards overlaps it; wait() makes the current stream wait for it."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist = dist
        self.group = group

    def all_reduce_start(self, t: torch.Tensor):
        return self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM, group=self.group, async_op=True)

    def wait(self, handle):
        handle.wait()


class _Clock:
    """Times the pieces of one rank: CUDA events on the current stream for device tensors, wall clock otherwise."""

    def __init__(self, on_device: bool):
        self.on_device = on_device
        self.marks = []

    def mark(self, label: str):
        if self.on_device:
            ev = torch.cuda.Event(enable_timing=True)
            ev.record()
            self.marks.append((label, ev))
        else:
            import time
            self.marks.append((label, time.perf_counter()))

    def spans(self) -> List[tuple]:
        """[(label of the piece that ended at the mark, milliseconds)] between consecutive marks."""
        if self.on_device:
            torch.cuda.synchronize()
        out = []
        for (_, a), (label, b) in zip(self.marks, self.marks[1:]):
            out.append((label, a.elapsed_time(b) if self.on_device else (b - a) * 1e3))
        return out


class BranchParallelPrefill:
    """One rank of a branch-parallel Kraken prefill.

    overlap=False waits for every all-reduce right where it is started (the blocking placement of a standard
    tensor-parallel layer): the difference to the default shows what the overlap hides.
    timing=True fills `last_timing` after every run: per layer the milliseconds of the attention half, of the
    time this rank's stream then still had to wait for the previous layer's all-reduce (what the attention half
    did NOT hide), and of the FFN half; plus the W_concat part with its blocking reduction and the head."""

    def __init__(self, engine, group, n_layer: int, overlap: bool = True, timing: bool = False):
        self.engine = engine
        self.group = group
        self.n_layer = n_layer
        self.overlap = overlap
        self.timing = timing
        self.last_timing = None

    def prefill(self, tokens: torch.Tensor) -> torch.Tensor:
        self.engine.stage_begin(tokens)
        return self._run()

    def decode_step(self, tokens: torch.Tensor) -> torch.Tensor:
        """One new token per sequence, after a prefill: the same order of pieces on [batch, d] tensors."""
        self.engine.stage_begin_decode(tokens)
        return self._run()

    def _run(self) -> torch.Tensor:
        e, g = self.engine, self.group
        x0, local_sum = e.stage_buffers()
        clock = _Clock(local_sum.is_cuda) if self.timing else None
        mark = clock.mark if clock else (lambda label: None)
        bufs = [torch.empty_like(local_sum), torch.empty_like(local_sum)]
        y, pending = x0, None                       # layer 1: the AllReduce is the identity (Algorithm 1)
        mark("start")
        for layer in range(self.n_layer):
            e.stage_attention(layer)                # overlaps the all-reduce started after the previous layer
            mark("attention")
            if pending is not None:
                g.wait(pending)
                pending = None
            mark("exposed_wait")
            e.stage_ffn(layer, y)
            if layer + 1 < self.n_layer:
                y = bufs[layer & 1]
                y.copy_(local_sum)                  # the next stage_ffn overwrites local_sum
                pending = g.all_reduce_start(y)
                if not self.overlap:
                    g.wait(pending)
                    pending = None
            mark("ffn")
        z = e.stage_concat()
        g.wait(g.all_reduce_start(z))               # nothing left to overlap: the logits need the full z
        mark("concat")
        logits = e.stage_head(z)
        mark("head")
        if clock:
            per = {"attention": [], "exposed_wait": [], "ffn": []}
            rest = {}
            for label, ms in clock.spans():
                if label in per:
                    per[label].append(ms)
                else:
                    rest[label] = ms
            self.last_timing = {"per_layer_ms": per, "concat_ms": rest.get("concat"), "head_ms": rest.get("head"),
                                "total_ms": sum(ms for _, ms in clock.spans()), "overlap": self.overlap}
        return logits


def lockstep_prefill(engines, n_layer: int, tokens: torch.Tensor, decode: bool = False) -> List[torch.Tensor]:
    """The same order of pieces as BranchParallelPrefill, for all ranks in one process: every piece is run for
    rank 0, 1, ... in turn and the all-reduce is an in-order sum (rank 0 first, the order in which a single
    device adds its branches).  decode: `tokens` is one new token per sequence after a prefill."""
    for e in engines:
        if decode:
            e.stage_begin_decode(tokens)
        else:
            e.stage_begin(tokens)
    bufs = [e.stage_buffers() for e in engines]
    ys = [x0 for x0, _ in bufs]
    for layer in range(n_layer):
        for e in engines:
            e.stage_attention(layer)
        for e, y in zip(engines, ys):
            e.stage_ffn(layer, y)
        if layer + 1 < n_layer:
            total = bufs[0][1].clone()
            for _, s in bufs[1:]:
                total = total + s
            ys = [total for _ in engines]
    zs = [e.stage_concat() for e in engines]
    z = zs[0].clone()
    for t in zs[1:]:
        z = z + t
    return [e.stage_head(z.clone()) for e in engines]
