"""The seeded generator: vectorised form equals the scalar definition, values have the stated law."""
import numpy as np
import torch

import kraken_inputs as ki


def test_vector_hash_equals_scalar_definition():
    for seed, tid, start in ((0, 0, 0), (1, 100, 5), (7, 10, (1 << 32) - 3), (3, 4, (1 << 33) + 11)):
        got = ki.hash32(seed, tid, start, 8, "cpu").tolist()
        ref = [ki.hash32_scalar(seed, tid, start + i) for i in range(8)]
        assert got == ref


def test_normal_table_is_the_quantile_function():
    bits = ki.normal_table_bits(0.02)
    vals = ki.bf16_bits_to_f32(bits)
    assert len(vals) == 65536
    assert np.all(np.diff(vals) >= 0)                       # quantiles are monotone
    assert np.array_equal(vals, -vals[::-1])                # symmetric law
    assert abs(vals[49152 + 0] - 0.02 * 0.6745) < 2e-4      # third quartile of N(0,1) is 0.6745
    assert 4.2 * 0.02 < vals[-1] < 4.4 * 0.02               # truncated near 4.3 sigma


def test_weights_and_tokens_law_and_reproducibility():
    s = ki.CONFIGS["C0"]
    w = ki.make_weights(s, seed=0)
    w2 = ki.make_weights(s, seed=0)
    for k in w:
        assert torch.equal(w[k], w2[k])
    assert not torch.equal(w["w_qkv"], ki.make_weights(s, seed=1)["w_qkv"])
    x = w["w_up"].float()
    assert abs(x.std().item() - 0.02) < 5e-4 and abs(x.mean().item()) < 1e-4
    assert torch.all(w["ln1_g"] == 1) and torch.all(w["ln2_b"] == 0) and torch.all(w["lnf_g"] == 1)
    assert ki.make_weights(s, bias=False)["b_qkv"] is None
    t = ki.uniform_tokens(1, s.vocab, 1, 128)
    assert t.dtype == torch.int32 and t.shape == (1, 128)
    assert int(t.min()) >= 0 and int(t.max()) < s.vocab
    big = ki.uniform_tokens(1, 50257, 4, 4096).double()
    assert abs(big.mean().item() / 50257 - 0.5) < 0.02
    # element i of a tensor depends only on (seed, tensor id, i): chunking does not matter
    a = ki.normal_bf16(3, 5, (1000,), chunk=64)
    b = ki.normal_bf16(3, 5, (1000,), chunk=1 << 20)
    assert torch.equal(a, b)


def test_flop_accounting():
    f = ki.algorithmic_flops(ki.CONFIGS["C3"])
    assert abs(f["gemm"] / 1e12 - 105.55) < 0.05 and abs(f["attn"] / 1e12 - 8.80) < 0.02
    # last-position logits only: the last layer's projections and FFN for the other T - B rows and its attention
    # for every query but the last are not needed (1/L of that work)
    s = ki.CONFIGS["C3"]
    g = ki.algorithmic_flops(s, last_positions_only=True)
    T, B, N, d, F, H, hd, l = s.batch * s.seqlen, s.batch, s.n_branch, s.d_model, s.d_ff, s.n_head, s.head_dim, s.seqlen
    assert f["gemm"] - g["gemm"] == 2.0 * (T - B) * N * (d * d + 2 * d * F)
    assert f["attn"] - g["attn"] == N * B * H * 4.0 * hd * (l * (l + 1) / 2 - l)
    assert g["tail"] == f["tail"] and 0.975 < g["total"] / f["total"] < 0.985
