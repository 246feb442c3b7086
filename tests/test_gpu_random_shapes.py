"""Seeded random shapes through the C ABI's step entry points, against the oracle's matching steps.

The hand-picked cases of test_gpu_ops.py sit on the tile boundaries someone thought of; these draw group counts, row
counts, widths, tile choices and epilogues at random (fixed seeds, so a failure reproduces), which is how ragged edges
in combinations nobody wrote down show up.  Integer-valued operands make the GEMM results exact.
"""
import numpy as np
import pytest
import torch

import kraken_inputs as ki
import oracle
import paper_2408_07802_b200 as kr

from test_gpu_ops import DEV, bf16_ulp_close, bits, gemm_case

pytestmark = pytest.mark.gpu

N_TILES = [0, 0, 0, 32, 64, 96, 128, 160, 192, 224, 256, 512]


@pytest.mark.parametrize("seed", range(24))
def test_gemm_random_shapes_integer_exact(seed):
    rng = np.random.default_rng(1000 + seed)
    G = int(rng.integers(1, 6))
    M = int(rng.choice([1, 7, 33, 64, 127, 128, 129, 255, 256, 257, 300, 511, 777, 1030]))
    n_out = 8 * int(rng.integers(1, 90))
    K = 8 * int(rng.integers(1, 70))
    n_tile = int(rng.choice(N_TILES))
    epi = int(rng.choice([kr.EPI_F32, kr.EPI_RESID_F32, kr.EPI_RESID_SUM]))
    wc = seed & 1        # odd seeds: W declared constant (its first tiles are requested before the predecessor ends)
    r = gemm_case(G, M, n_out, K, epi, n_tile, seed=seed, integer=True, w_constant=wc)
    what = (G, M, n_out, K, epi, n_tile, wc)
    assert np.array_equal(r["out_f32"], r["ref"]), what
    if epi == kr.EPI_RESID_SUM:
        assert np.array_equal(r["sum"], r["ref"].sum(0)), what


@pytest.mark.parametrize("seed", range(12))
def test_gemm_random_shapes_bf16_epilogues(seed):
    rng = np.random.default_rng(2000 + seed)
    G = int(rng.integers(1, 5))
    M = int(rng.choice([5, 96, 128, 200, 384, 640]))
    n_out = 8 * int(rng.integers(4, 70))
    K = 8 * int(rng.integers(8, 60))
    n_tile = int(rng.choice(N_TILES))
    epi = int(rng.choice([kr.EPI_BF16, kr.EPI_GELU_BF16]))
    r = gemm_case(G, M, n_out, K, epi, n_tile, seed=seed, w_constant=seed & 1)
    ok, worst = bf16_ulp_close(r["out_bf16"], r["ref"], ulps=1.0, atol=3e-4)
    assert ok, ((G, M, n_out, K, epi, n_tile), worst)


@pytest.mark.parametrize("seed", range(16))
def test_attention_random_shapes(seed):
    rng = np.random.default_rng(3000 + seed)
    hd = int(rng.choice([64, 72, 96, 104, 128]))
    Hkv = int(rng.choice([1, 2, 3]))
    rep = int(rng.choice([1, 1, 2, 4]))
    H = Hkv * rep
    G = int(rng.integers(1, 4))
    B = int(rng.integers(1, 4))
    seqlen = int(rng.choice([1, 17, 128, 129, 255, 256, 257, 400, 513, 900]))
    pos0 = int(rng.choice([0, 0, 0, 5, 128, 300]))
    P = pos0 + seqlen + int(rng.integers(0, 40))
    d = H * hd
    q = ki.normal_bf16(seed, 0, (G, B * seqlen, d), 1.0, DEV)
    kc = ki.normal_bf16(seed, 1, (G, B, Hkv, P, hd), 1.0, DEV)
    vc = ki.normal_bf16(seed, 2, (G, B, Hkv, P, hd), 1.0, DEV)
    kc[:, :, :, pos0 + seqlen:] = float("nan")      # rows past the sequence must not leak
    vc[:, :, :, pos0 + seqlen:] = float("nan")
    out = kr.op_attention(q, kc, vc, B, seqlen, pos0, H).float().cpu().numpy()
    what = (G, B, H, Hkv, hd, seqlen, pos0, P)
    assert not np.isnan(out).any(), what
    qn, kn, vn = q.float().cpu().numpy(), kc.float().cpu().numpy(), vc.float().cpu().numpy()
    for g, b, h in {(0, 0, 0), (G - 1, B - 1, H - 1), (G // 2, B // 2, H // 2)}:
        ref = oracle.attention_head(qn[g, b * seqlen:(b + 1) * seqlen, h * hd:(h + 1) * hd],
                                    kn[g, b, h // rep, :pos0 + seqlen], vn[g, b, h // rep, :pos0 + seqlen], q_pos0=pos0)
        got = out[g, b * seqlen:(b + 1) * seqlen, h * hd:(h + 1) * hd]
        assert np.abs(got - ref).max() < 3e-2, (what, g, b, h, np.abs(got - ref).max())


@pytest.mark.parametrize("seed", range(16))
def test_layernorm_random_shapes(seed):
    rng = np.random.default_rng(4000 + seed)
    G = int(rng.integers(1, 10))
    d = 4 * int(rng.choice([8, 65, 192, 256, 312, 480, 512, 624, 780, 1024, 1248, 1856, 2048]))
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    rows = int(rng.choice([1, 5, 31, 130, 3 * sms + 1, 8 * sms + 5, 9 * sms]))
    if G * rows * d > 60_000_000:
        rows = max(1, 60_000_000 // (G * d))
    with_y = bool(rng.integers(0, 2))
    with_status = bool(rng.integers(0, 2))
    a = (ki.normal_bf16(seed, 0, (G, rows, d), 1.0, DEV).float() * 1.1 + 0.2).contiguous()
    y = ki.normal_bf16(seed, 1, (rows, d), 1.5, DEV).float().contiguous() if with_y else None
    gamma = (1 + ki.normal_bf16(seed, 2, (G, d), 0.3, DEV).float()).to(torch.bfloat16)
    beta = ki.normal_bf16(seed, 3, (G, d), 0.3, DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV) if with_status else None
    out = kr.op_layernorm(a, y, gamma, beta, status=status)
    torch.cuda.synchronize()
    if status is not None:
        assert int(status.item()) == 0
    pick = sorted({0, rows // 2, rows - 1})
    for g in {0, G - 1}:
        ref = oracle.layernorm(a[g][pick].cpu().numpy(), None if y is None else y[pick].cpu().numpy(),
                               bits(gamma[g]), bits(beta[g]))
        ok, worst = bf16_ulp_close(out[g][pick].float().cpu().numpy(), ref, ulps=1.0, atol=1e-5)
        assert ok, ((G, rows, d, with_y, with_status), g, worst)


@pytest.mark.parametrize("seed", range(16))
def test_decode_attention_random_shapes(seed):
    rng = np.random.default_rng(5000 + seed)
    hd = int(rng.choice([64, 72, 96, 104, 128]))
    Hkv = int(rng.choice([1, 2, 3]))
    rep = int(rng.choice([1, 1, 2, 4, 8]))
    H = Hkv * rep
    G = int(rng.integers(1, 4))
    B = int(rng.integers(1, 6))
    n_keys = int(rng.choice([1, 2, 63, 64, 65, 300, 1000, 2500]))
    splits = int(rng.choice([0, 0, 1, 2, 5]))
    P = n_keys + int(rng.integers(0, 20))
    d = H * hd
    q = ki.normal_bf16(seed, 0, (G, B, d), 1.0, DEV)
    kc = ki.normal_bf16(seed, 1, (G, B, Hkv, P, hd), 1.0, DEV)
    vc = ki.normal_bf16(seed, 2, (G, B, Hkv, P, hd), 1.0, DEV)
    kc[:, :, :, n_keys:] = float("nan")
    vc[:, :, :, n_keys:] = float("nan")
    sp, nb = kr.decode_attention_sizes(G, B, n_keys, H, hd, splits)
    part = torch.empty(max(nb, 16), dtype=torch.uint8, device=DEV)
    out = kr.op_decode_attention(q, kc, vc, n_keys, sp, part).float().cpu().numpy()
    what = (G, B, H, Hkv, hd, n_keys, splits, sp)
    assert not np.isnan(out).any(), what
    qn, kn, vn = q.float().cpu().numpy(), kc.float().cpu().numpy(), vc.float().cpu().numpy()
    for g, b, h in {(0, 0, 0), (G - 1, B - 1, H - 1), (G // 2, B // 2, H // 2)}:
        ref = oracle.attention_head(qn[g, b:b + 1, h * hd:(h + 1) * hd], kn[g, b, h // rep, :n_keys],
                                    vn[g, b, h // rep, :n_keys], q_pos0=n_keys - 1)
        got = out[g, b, h * hd:(h + 1) * hd]
        assert np.abs(got - ref[0]).max() < 3e-2, (what, g, b, h, np.abs(got - ref[0]).max())


@pytest.mark.parametrize("seed", range(10))
def test_whole_model_random_configurations(seed):
    """Random small models (branches, layers, head dim, key/value heads, FFN width, vocabulary, variant) and request
    shapes: logits at every position against the oracle, then two decode steps."""
    from test_gpu_model import REL_L2_MAX, MAX_ABS_MAX, build, check_parity, host_bits, logits_metrics, oracle_all_logits
    rng = np.random.default_rng(6000 + seed)
    hd = int(rng.choice([64, 72, 96, 104, 128]))
    Hkv = int(rng.choice([1, 2]))
    rep = int(rng.choice([1, 2, 3]))
    H = Hkv * rep
    variant = int(rng.choice([0, 0, 1, 2]))
    batch = int(rng.integers(1, 4))
    seqlen = int(rng.choice([1, 9, 64, 130, 257, 300]))
    s = ki.KrakenShape(f"R{seed}", int(rng.integers(1, 6)), int(rng.integers(1, 4)), H * hd, H, 8 * int(rng.integers(8, 64)),
                       int(rng.integers(100, 700)), seqlen + 8, batch, seqlen, n_kv_head=0 if rep == 1 else Hkv,
                       no_combine=int(variant != 0), parallel_ffn=int(variant == 2))   # the parallel variant has no cross-branch term
    m, w = build(s)
    wb = host_bits(w)
    steps = 2
    tok = ki.uniform_tokens(seed, s.vocab, batch, seqlen + steps, DEV)
    first = tok[:, :seqlen].contiguous()
    got_all = m.prefill_all_logits(first).cpu().numpy()
    orcs = []
    for b in range(batch):
        ids = tok[b, :seqlen].cpu().numpy()
        ref32, orc = oracle_all_logits(s, wb, ids, False)
        refbf, _ = oracle_all_logits(s, wb, ids, True)
        check_parity(got_all[b], ref32, refbf, f"{s} seq {b}")
        orcs.append(orc)
    assert m.device_status() == 0
    for t in range(steps):
        got = m.decode_step(tok[:, seqlen + t].contiguous()).cpu().numpy()
        for b in range(batch):
            ref = orcs[b].decode_step(int(tok[b, seqlen + t]))
            rel, mx = logits_metrics(got[b], ref)
            assert rel <= REL_L2_MAX and mx <= MAX_ABS_MAX, (s, t, b, rel, mx)
    assert m.device_status() == 0 and m.cur_len == seqlen + steps
    m.close()


@pytest.mark.parametrize("seed", range(6))
def test_packed_prefill_random_lengths(seed):
    """Packed (ragged) batches with random numbers of sequences and random lengths, then ragged decode steps."""
    from test_gpu_model import test_packed_prefill_and_ragged_decode as packed_case
    rng = np.random.default_rng(7000 + seed)
    name = str(rng.choice(["C0", "K0-104", "C0-gqa", "K0-72"]))
    s = ki.CONFIGS[name]
    lens = [int(x) for x in rng.integers(1, s.max_pos - 5, size=int(rng.integers(1, 7)))]
    packed_case(name, lens)
