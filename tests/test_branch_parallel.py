"""Branch-parallel prefill (one rank per group of branches, the cross-branch sum an all-reduce).

CPU: the ordering of pieces and collectives in `BranchParallelPrefill`, run as two gloo ranks whose "engine"
is built from the oracle's single steps, against the oracle's whole-model forward pass.
GPU: the library's stage calls, with several ranks standing in one process on one GPU and driven in lockstep
(no kernel ever waits for another rank), against the ordinary single-GPU prefill of the same model and against
the oracle's logits.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

import kraken_inputs as ki
import oracle
from paper_2408_07802_b200 import branch_parallel as bp


def bits(t):
    return None if t is None else ki.bf16_tensor_to_bits(t)


class OracleStageEngine:
    """The stage interface of one rank on CPU tensors, every step a call of the oracle's single-step routines
    (one sequence).  Test infrastructure: it exists to exercise the ordering logic under a real collective."""

    def __init__(self, shape, w):
        self.s, self.w = shape, w
        self.N = w["ln1_g"].shape[1]

    def stage_begin(self, tokens):
        ids = tokens[0].numpy()
        self.l = len(ids)
        wte, wpe = self.w["wte"].float().numpy(), self.w["wpe"].float().numpy()
        self.x0 = torch.from_numpy(wte[ids] + wpe[: self.l])
        self.x = [self.x0.clone() for _ in range(self.N)]
        self.local_sum = torch.zeros_like(self.x0)

    def stage_buffers(self):
        return self.x0, self.local_sum

    def stage_attention(self, layer):
        s, w, H, hd = self.s, self.w, self.s.n_head, self.s.head_dim
        d = s.d_model
        self.a = []
        for n in range(self.N):
            u = oracle.layernorm(self.x[n].numpy(), None, bits(w["ln1_g"][layer, n]), bits(w["ln1_b"][layer, n]))
            qkv = oracle.linear(u, bits(w["w_qkv"][layer, n]), bits(w["b_qkv"][layer, n]))
            o = np.empty((self.l, d), dtype=np.float32)
            for h in range(H):
                o[:, h * hd:(h + 1) * hd] = oracle.attention_head(qkv[:, h * hd:(h + 1) * hd],
                                                                  qkv[:, d + h * hd:d + (h + 1) * hd],
                                                                  qkv[:, 2 * d + h * hd:2 * d + (h + 1) * hd])
            proj = oracle.linear(o, bits(w["w_proj"][layer, n]), bits(w["b_proj"][layer, n]))
            self.a.append(self.x[n].numpy() + proj)

    def stage_ffn(self, layer, y):
        w = self.w
        for n in range(self.N):
            hh = oracle.layernorm(self.a[n], y.numpy(), bits(w["ln2_g"][layer, n]), bits(w["ln2_b"][layer, n]))
            g = oracle.linear(hh, bits(w["w_up"][layer, n]), bits(w["b_up"][layer, n]))
            g = np.vectorize(oracle.gelu, otypes=[np.float32])(g)
            out = self.a[n] + oracle.linear(g, bits(w["w_down"][layer, n]), bits(w["b_down"][layer, n]))
            self.x[n] = torch.from_numpy(out)
        self.local_sum.copy_(torch.stack(self.x).sum(0))

    def stage_concat(self):
        cat = torch.cat([x[-1:] for x in self.x], dim=1).numpy()
        return torch.from_numpy(oracle.linear(cat, bits(self.w["w_concat"]), bits(self.w["b_concat"])))

    def stage_head(self, z):
        zf = oracle.layernorm(z.numpy(), None, bits(self.w["lnf_g"]), bits(self.w["lnf_b"]))
        return torch.from_numpy(oracle.linear(zf, bits(self.w["wte"])))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


SHAPE = ki.KrakenShape("bp", 4, 3, 32, 2, 64, 97, 24, 1, 10)
SPLIT = [(0, 3), (3, 1)]          # rank 0 holds three branches, rank 1 one


def _worker(rank, world, port, out):
    import torch.distributed as dist
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = ki.make_weights(SHAPE, seed=5, std=0.08)
    first, count = SPLIT[rank]
    mine = bp.slice_weights(w, SHAPE.n_branch, first, count, with_concat_bias=rank == 0)
    eng = OracleStageEngine(SHAPE, mine)
    tok = ki.uniform_tokens(8, SHAPE.vocab, 1, SHAPE.seqlen)
    runner = bp.BranchParallelPrefill(eng, bp.TorchDistGroup(), SHAPE.n_layer, timing=True)
    logits = runner.prefill(tok)
    out[rank] = logits.numpy()
    t = runner.last_timing
    assert len(t["per_layer_ms"]["attention"]) == SHAPE.n_layer and t["total_ms"] > 0 and t["overlap"]
    # the blocking placement of the all-reduce gives the same logits (same sums in the same order)
    blocking = bp.BranchParallelPrefill(eng, bp.TorchDistGroup(), SHAPE.n_layer, overlap=False).prefill(tok)
    assert np.array_equal(blocking.numpy(), out[rank])
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_with_oracle_engines_equal_the_whole_model():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    w = ki.make_weights(SHAPE, seed=5, std=0.08)
    tok = ki.uniform_tokens(8, SHAPE.vocab, 1, SHAPE.seqlen)
    ref, _ = oracle.Oracle(SHAPE, {k: bits(v) for k, v in w.items()}).prefill(tok[0].numpy(), logits_from=SHAPE.seqlen - 1)
    for rank in range(world):
        assert np.max(np.abs(res[rank][0] - ref[0])) < 2e-5 * max(1.0, np.abs(ref).max()), rank
    assert np.array_equal(res[0], res[1])            # every rank ends with the same logits


def test_slice_weights_partitions_the_model():
    w = ki.make_weights(SHAPE, seed=5)
    parts = [bp.slice_weights(w, 4, f, c, with_concat_bias=f == 0) for f, c in SPLIT]
    assert torch.equal(torch.cat([p["w_up"] for p in parts], dim=1), w["w_up"])
    d = SHAPE.d_model
    assert torch.equal(torch.cat([p["w_concat"] for p in parts], dim=1), w["w_concat"])
    assert parts[0]["w_concat"].shape == (d, 3 * d) and parts[1]["b_concat"] is None
    assert parts[0]["wte"] is w["wte"]


@pytest.mark.gpu
@pytest.mark.parametrize("name,split", [("C0", [(0, 1), (1, 1)]), ("K0-96", [(0, 1), (1, 1), (2, 1), (3, 1)]),
                                        ("K0-96", [(0, 3), (3, 1)]), ("C0", [(0, 2)])])
def test_stage_calls_in_lockstep_equal_the_single_gpu_prefill(name, split):
    import paper_2408_07802_b200 as kr
    dev = "cuda:0"
    s = ki.CONFIGS[name]
    w = ki.make_weights(s, seed=0, device=dev)
    whole = kr.KrakenModel(kr.make_config(s), w, dev)
    l0 = min(s.seqlen, s.max_pos - 4)               # room for the decode steps below
    tok = ki.uniform_tokens(2, s.vocab, s.batch, l0, dev)
    # the pieces run every layer on every row; so does the reference (the single call's shortcut for the last layer's
    # other rows takes other kernels for the last positions)
    with kr.tuning(kr.TUNE_LAST_LAYER, 1):
        ref = whole.prefill(tok)
    engines = []
    for first, count in split:
        mine = bp.slice_weights(w, s.n_branch, first, count, with_concat_bias=first == 0)
        engines.append(kr.KrakenModel(kr.make_config(s, n_branch=count), mine, dev))
    outs = bp.lockstep_prefill(engines, s.n_layer, tok)
    for o in outs:
        err = (o - ref).abs().max().item()
        assert err <= 2e-3 * max(1.0, ref.abs().max().item()), err
    # and against the oracle's whole-model forward pass, within the bounds stated for the logits
    wb = {k: bits(v) for k, v in w.items()}
    orcs = []
    for b in range(s.batch):
        orc = oracle.Oracle(s, wb)
        want, _ = orc.prefill(tok[b].cpu().numpy(), logits_from=l0 - 1)
        orcs.append(orc)
        for o in outs:
            got = o[b].float().cpu().numpy()
            assert np.linalg.norm(got - want[0]) / np.linalg.norm(want[0]) <= 1e-2
            assert np.abs(got - want[0]).max() <= 5e-2
    # every rank's cache holds exactly its branches' rows of the whole model's cache
    for (first, count), e in zip(split, engines):
        assert e.cur_len == l0 and e.device_status() == 0
        for n in range(count):
            for which in (0, 1):
                a = e.kv_view(s.n_layer - 1, n, which)[:, :, :l0].float()
                b = whole.kv_view(s.n_layer - 1, first + n, which)[:, :, :l0].float()
                assert (a - b).abs().max().item() <= 2.0 ** -6 * b.abs().max().item()
    # decode steps driven the same way continue from the caches
    nxt = ki.uniform_tokens(3, s.vocab, 1, s.batch, dev)[0].contiguous()
    for step in range(2):
        want = whole.decode_step(nxt)
        outs = bp.lockstep_prefill(engines, s.n_layer, nxt, decode=True)
        for o in outs:
            err = (o - want).abs().max().item()
            assert err <= 2e-3 * max(1.0, want.abs().max().item()), (step, err)
        for b in range(s.batch):
            truth = orcs[b].decode_step(int(nxt[b]))
            got = outs[0][b].float().cpu().numpy()
            assert np.linalg.norm(got - truth) / np.linalg.norm(truth) <= 1e-2, (step, b)
            assert np.abs(got - truth).max() <= 5e-2, (step, b)
    assert all(e.cur_len == l0 + 2 for e in engines)
    # out-of-order calls are refused
    with pytest.raises(kr.KrakenError) as ex:
        engines[0].stage_attention(1)
    assert ex.value.status == kr.ESTATE
    for e in engines:
        e.close()
    whole.close()


@pytest.mark.gpu
def test_one_nccl_rank_through_the_collective_path_equals_prefill():
    """BranchParallelPrefill with torch.distributed's NCCL backend (a group of one rank, all this run has): the
    asynchronous all-reduce and the waits are the real ones, and a rank that holds every branch must reproduce
    the ordinary prefill."""
    import torch.distributed as dist
    import paper_2408_07802_b200 as kr
    dev = "cuda:0"
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{_free_port()}", rank=0, world_size=1)
    try:
        s = ki.CONFIGS["C1"]
        w = ki.make_weights(s, seed=0, device=dev)
        m = kr.KrakenModel(kr.make_config(s), w, dev)
        tok = ki.uniform_tokens(2, s.vocab, s.batch, s.seqlen, dev)
        with kr.tuning(kr.TUNE_LAST_LAYER, 1):   # every layer on every row, like the pieces
            ref = m.prefill(tok).clone()
        runner = bp.BranchParallelPrefill(m, bp.TorchDistGroup(), s.n_layer, timing=True)
        got = runner.prefill(tok)
        t = runner.last_timing
        assert len(t["per_layer_ms"]["ffn"]) == s.n_layer and all(v >= 0 for v in t["per_layer_ms"]["exposed_wait"])
        torch.cuda.synchronize()
        err = (got - ref).abs().max().item()
        assert err <= 2e-3 * max(1.0, ref.abs().max().item()), err
        assert m.cur_len == s.seqlen and m.device_status() == 0
        m.close()
    finally:
        dist.destroy_process_group()

