"""Pins of the CPU oracle against what the paper and the mathematics fix.

Each test checks the oracle against something other than itself: closed forms,
brute force on tiny inputs, special cases that reduce to library routines,
invariants (causality, branch permutation, prefill + decode = longer prefill),
and the parameter counts the paper prints.
"""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import kraken_inputs as ki
import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bits(t):
    return None if t is None else ki.bf16_tensor_to_bits(t)


def wbits(w):
    return {k: bits(v) for k, v in w.items()}


def small_shape(**kw):
    base = dict(name="S", n_branch=3, n_layer=2, d_model=32, n_head=2, d_ff=64, vocab=97, max_pos=24,
                batch=1, seqlen=12)
    base.update(kw)
    return ki.KrakenShape(**base)


def rand_weights(shape, seed=3, std=0.08, ln_random=True, bias=True):
    """Weights with non-trivial LayerNorm parameters so gamma/beta handling is exercised."""
    w = ki.make_weights(shape, seed=seed, std=std, bias=bias)
    if ln_random:
        for i, k in enumerate(("ln1_g", "ln2_g", "lnf_g")):
            w[k] = (1.0 + ki.normal_bf16(seed, 40 + i, w[k].shape, 0.2).float()).to(torch.bfloat16)
        for i, k in enumerate(("ln1_b", "ln2_b", "lnf_b")):
            w[k] = ki.normal_bf16(seed, 50 + i, w[k].shape, 0.2)
    return w


# ------------------------------------------------------------------ scalar steps

def test_gelu_closed_forms():
    assert oracle.gelu(0.0) == 0.0
    # Phi(1) = 0.841344746..., so GELU(1) = Phi(1)
    assert abs(oracle.gelu(1.0) - 0.8413447460685429) < 1e-7
    assert abs(oracle.gelu(-1.0) + 0.15865525393145707) < 1e-7
    for x in (0.1, 0.7, 1.3, 2.9, 5.0):
        # Phi(x) + Phi(-x) = 1  =>  GELU(x) - GELU(-x) = x
        assert abs(oracle.gelu(x) - oracle.gelu(-x) - x) < 1e-6
    assert abs(oracle.gelu(12.0) - 12.0) < 1e-6
    assert abs(oracle.gelu(-12.0)) < 1e-6
    xs = np.linspace(-6, 6, 1201)
    diff = max(abs(oracle.gelu(float(x)) - oracle.gelu(float(x), True)) for x in xs)
    assert 1e-5 < diff < 1e-3  # the two variants differ, but only slightly
    ref = F.gelu(torch.tensor(xs, dtype=torch.float64)).numpy()
    got = np.array([oracle.gelu(float(x)) for x in xs])
    assert np.max(np.abs(got - ref)) < 1e-6


def test_round_bf16_ties_to_even():
    # 1 + 2^-8 is exactly half-way between bf16 neighbours 1 and 1 + 2^-7 -> even (1.0)
    assert oracle.round_bf16(1.0 + 2 ** -8) == 1.0
    # 1 + 3*2^-8 is half-way between 1 + 2^-7 and 1 + 2^-6 -> even mantissa (1 + 2^-6)
    assert oracle.round_bf16(1.0 + 3 * 2 ** -8) == 1.0 + 2 ** -6
    assert oracle.round_bf16(1.0 + 2 ** -8 + 2 ** -20) == 1.0 + 2 ** -7
    x = np.random.default_rng(0).standard_normal(1000).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).float().numpy()
    got = np.array([oracle.round_bf16(float(v)) for v in x], dtype=np.float32)
    assert np.array_equal(ref, got)
    assert np.array_equal(ki.bf16_bits_to_f32(ki.f32_to_bf16_bits(x)), ref)


def test_layernorm_closed_forms():
    d = 16
    g = ki.f32_to_bf16_bits(np.linspace(0.5, 2.0, d).astype(np.float32))
    b = ki.f32_to_bf16_bits(np.linspace(-1.0, 1.0, d).astype(np.float32))
    gf, bf = ki.bf16_bits_to_f32(g), ki.bf16_bits_to_f32(b)
    const = np.full((1, d), 3.25, dtype=np.float32)
    out = oracle.layernorm(const, None, g, b)
    assert np.allclose(out[0], bf, atol=1e-6)  # zero variance: only beta survives
    alt = np.array([[(-1.0) ** j for j in range(d)]], dtype=np.float32)
    eps = 1e-5
    out = oracle.layernorm(alt, None, g, b, eps=eps)
    assert np.allclose(out[0], alt[0] * gf / math.sqrt(1 + eps) + bf, atol=1e-6)
    # the optional second operand is added before normalisation
    out2 = oracle.layernorm(alt * 0.25, alt * 0.75, g, b, eps=eps)
    assert np.allclose(out, out2, atol=1e-6)


def test_layernorm_matches_library():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((7, 48)).astype(np.float32) * 3 + 1
    g = ki.f32_to_bf16_bits(rng.standard_normal(48).astype(np.float32))
    b = ki.f32_to_bf16_bits(rng.standard_normal(48).astype(np.float32))
    ref = F.layer_norm(torch.from_numpy(x).double(), (48,), torch.from_numpy(ki.bf16_bits_to_f32(g)).double(),
                       torch.from_numpy(ki.bf16_bits_to_f32(b)).double(), 1e-5).numpy()
    got = oracle.layernorm(x, None, g, b)
    assert np.max(np.abs(got - ref)) < 1e-5
    rounded = oracle.layernorm(x, None, g, b, round_out=True)
    assert np.array_equal(rounded, torch.from_numpy(got).to(torch.bfloat16).float().numpy())


def test_linear_orientation_and_values():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((5, 12)).astype(np.float32)
    # weight [n_out, n_in] that picks input feature sel[o] for output o: any transposition fails
    sel = [3, 11, 0, 7, 7, 2, 9]
    W = np.zeros((len(sel), 12), dtype=np.float32)
    for o, i in enumerate(sel):
        W[o, i] = 1.0
    bias = np.arange(len(sel), dtype=np.float32)
    out = oracle.linear(x, ki.f32_to_bf16_bits(W), ki.f32_to_bf16_bits(bias))
    assert np.array_equal(out, x[:, sel] + bias)
    Wr = ki.f32_to_bf16_bits(rng.standard_normal((9, 12)).astype(np.float32))
    br = ki.f32_to_bf16_bits(rng.standard_normal(9).astype(np.float32))
    ref = x.astype(np.float64) @ ki.bf16_bits_to_f32(Wr).astype(np.float64).T + ki.bf16_bits_to_f32(br)
    assert np.max(np.abs(oracle.linear(x, Wr, br) - ref)) < 1e-5
    assert np.max(np.abs(oracle.linear(x, Wr) - (ref - ki.bf16_bits_to_f32(br)))) < 1e-5


def brute_attention(q, k, v, q_pos0=0):
    n_q, hd = q.shape
    out = np.zeros((n_q, hd))
    for i in range(n_q):
        p = q_pos0 + i
        s = [sum(float(q[i, c]) * float(k[j, c]) for c in range(hd)) / math.sqrt(hd) for j in range(p + 1)]
        m = max(s)
        e = [math.exp(v_ - m) for v_ in s]
        z = sum(e)
        for j in range(p + 1):
            for c in range(hd):
                out[i, c] += e[j] / z * float(v[j, c])
    return out


def test_attention_brute_force_and_closed_forms():
    rng = np.random.default_rng(3)
    l, hd = 9, 8
    q = rng.standard_normal((l, hd)).astype(np.float32) * 2
    k = rng.standard_normal((l, hd)).astype(np.float32) * 2
    v = rng.standard_normal((l, hd)).astype(np.float32)
    got = oracle.attention_head(q, k, v)
    assert np.max(np.abs(got - brute_attention(q, k, v))) < 1e-6
    # zero queries: uniform weights over the visible prefix -> running mean of v
    got0 = oracle.attention_head(np.zeros_like(q), k, v)
    run = np.cumsum(v.astype(np.float64), axis=0) / np.arange(1, l + 1)[:, None]
    assert np.max(np.abs(got0 - run)) < 1e-6
    # a single position attends only to itself
    assert np.allclose(oracle.attention_head(q[:1], k[:1], v[:1]), v[:1], atol=1e-7)
    # library routine
    ref = F.scaled_dot_product_attention(torch.from_numpy(q).double()[None], torch.from_numpy(k).double()[None],
                                         torch.from_numpy(v).double()[None], is_causal=True)[0].numpy()
    assert np.max(np.abs(got - ref)) < 1e-6
    # queries that start at an offset (decode): rows of the full result
    tail = oracle.attention_head(q[6:], k, v, q_pos0=6)
    assert np.max(np.abs(tail - got[6:])) < 1e-7
    # a huge score on a masked (future) key must not leak
    k2 = k.copy()
    k2[5] = q[2] * 50
    leak = oracle.attention_head(q, k2, v)
    assert np.array_equal(leak[:5], got[:5])


# ------------------------------------------------------------------ library composition

def torch_kraken(shape, w, ids, y_zero=False, final_ln=True):
    """Kraken forward composed from torch CPU library routines in fp64 (all positions)."""
    W = {k: (None if v is None else v.double()) for k, v in w.items()}
    N, L, d, H = shape.n_branch, shape.n_layer, shape.d_model, shape.n_head
    hd = d // H
    l = len(ids)
    idt = torch.as_tensor(ids, dtype=torch.long)
    x0 = W["wte"][idt] + W["wpe"][:l]
    xs = [x0.clone() for _ in range(N)]
    for layer in range(L):
        y = x0 if layer == 0 else torch.stack(xs).sum(0)
        if y_zero:
            y = torch.zeros_like(x0)
        nxt = []
        for n in range(N):
            u = F.layer_norm(xs[n], (d,), W["ln1_g"][layer, n], W["ln1_b"][layer, n], shape.ln_eps)
            qkv = F.linear(u, W["w_qkv"][layer, n], None if W["b_qkv"] is None else W["b_qkv"][layer, n])
            q, k, v = [t.reshape(l, H, hd).transpose(0, 1) for t in qkv.split(d, dim=1)]
            o = F.scaled_dot_product_attention(q[None], k[None], v[None], is_causal=True)[0]
            o = o.transpose(0, 1).reshape(l, d)
            a = xs[n] + F.linear(o, W["w_proj"][layer, n], None if W["b_proj"] is None else W["b_proj"][layer, n])
            hh = F.layer_norm(a + y, (d,), W["ln2_g"][layer, n], W["ln2_b"][layer, n], shape.ln_eps)
            g = F.gelu(F.linear(hh, W["w_up"][layer, n], None if W["b_up"] is None else W["b_up"][layer, n]))
            nxt.append(a + F.linear(g, W["w_down"][layer, n], None if W["b_down"] is None else W["b_down"][layer, n]))
        xs = nxt
    z = F.linear(torch.cat(xs, dim=1), W["w_concat"], W["b_concat"])
    if final_ln:
        z = F.layer_norm(z, (d,), W["lnf_g"], W["lnf_b"], shape.ln_eps)
    return (z @ W["wte"].T).numpy(), [x.numpy() for x in xs]


def test_single_branch_reduces_to_gpt2_stack():
    """N = 1 with the y term dropped and W_concat = I is a pre-LN GPT-2 block stack."""
    shape = small_shape(n_branch=1, n_layer=3)
    w = rand_weights(shape)
    w["w_concat"] = torch.eye(shape.d_model, dtype=torch.bfloat16)
    w["b_concat"] = None
    ids = ki.uniform_tokens(5, shape.vocab, 1, shape.seqlen)[0].numpy()

    # plain GPT-2 style stack from library routines, written without any Kraken notion
    W = {k: (None if v is None else v.double()) for k, v in w.items()}
    d, H = shape.d_model, shape.n_head
    l = len(ids)
    x = W["wte"][torch.as_tensor(ids, dtype=torch.long)] + W["wpe"][:l]
    for layer in range(shape.n_layer):
        u = F.layer_norm(x, (d,), W["ln1_g"][layer, 0], W["ln1_b"][layer, 0], 1e-5)
        qkv = F.linear(u, W["w_qkv"][layer, 0], W["b_qkv"][layer, 0])
        q, k, v = [t.reshape(l, H, d // H).transpose(0, 1) for t in qkv.split(d, dim=1)]
        o = F.scaled_dot_product_attention(q[None], k[None], v[None], is_causal=True)[0].transpose(0, 1).reshape(l, d)
        x = x + F.linear(o, W["w_proj"][layer, 0], W["b_proj"][layer, 0])
        hh = F.layer_norm(x, (d,), W["ln2_g"][layer, 0], W["ln2_b"][layer, 0], 1e-5)
        x = x + F.linear(F.gelu(F.linear(hh, W["w_up"][layer, 0], W["b_up"][layer, 0])),
                         W["w_down"][layer, 0], W["b_down"][layer, 0])
    ref = (F.layer_norm(x, (d,), W["lnf_g"], W["lnf_b"], 1e-5) @ W["wte"].T).numpy()

    orc = oracle.Oracle(shape, wbits(w), y_zero=True)
    got, _ = orc.prefill(ids)
    assert np.max(np.abs(got - ref)) < 2e-5 * max(1.0, np.max(np.abs(ref)))


@pytest.mark.parametrize("final_ln", [True, False])
def test_matches_library_composition(final_ln):
    shape = small_shape()
    w = rand_weights(shape)
    ids = ki.uniform_tokens(7, shape.vocab, 1, shape.seqlen)[0].numpy()
    ref, ref_x = torch_kraken(shape, w, ids, final_ln=final_ln)
    orc = oracle.Oracle(shape, wbits(w), final_ln=final_ln)
    got, lo = orc.prefill(ids, want_layer_out=True)
    assert np.max(np.abs(got - ref)) < 2e-5 * max(1.0, np.max(np.abs(ref)))
    for n in range(shape.n_branch):
        assert np.max(np.abs(lo[-1, n] - ref_x[n])) < 2e-5


@pytest.mark.parametrize("d_model,n_head", [(144, 2), (208, 2), (96, 1)])
def test_engine_head_dims_match_library_composition(d_model, n_head):
    """Head dims of the paper's engine shapes (Table 3: 72, 104, 96) with the 2 d FFN: the oracle against the
    same composition written with library routines."""
    shape = small_shape(d_model=d_model, n_head=n_head, d_ff=2 * d_model, n_branch=2)
    w = rand_weights(shape)
    ids = ki.uniform_tokens(11, shape.vocab, 1, shape.seqlen)[0].numpy()
    ref, _ = torch_kraken(shape, w, ids, final_ln=True)
    got, _ = oracle.Oracle(shape, wbits(w)).prefill(ids)
    assert np.max(np.abs(got - ref)) < 2e-5 * max(1.0, np.max(np.abs(ref)))


def test_c0_matches_library_composition():
    shape = ki.CONFIGS["C0"]
    w = ki.make_weights(shape, seed=0)
    ids = ki.uniform_tokens(1, shape.vocab, 1, 48)[0].numpy()
    ref, _ = torch_kraken(shape, w, ids)
    got, _ = oracle.Oracle(shape, wbits(w)).prefill(ids)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 1e-5


# ------------------------------------------------------------------ the cross-branch combination

def sublayer_from_steps(shape, w, layer, n, x_n, y):
    """Algorithm 1 for one sub-layer, assembled from the individually pinned step functions."""
    d, H = shape.d_model, shape.n_head
    hd = d // H
    g = lambda k: bits(w[k][layer, n])
    u = oracle.layernorm(x_n, None, g("ln1_g"), g("ln1_b"))
    qkv = oracle.linear(u, g("w_qkv"), g("b_qkv"))
    o = np.zeros_like(x_n)
    for h in range(H):
        sl = slice(h * hd, (h + 1) * hd)
        o[:, sl] = oracle.attention_head(qkv[:, sl], qkv[:, d:2 * d][:, sl], qkv[:, 2 * d:][:, sl])
    a = x_n + oracle.linear(o, g("w_proj"), g("b_proj"))
    hh = oracle.layernorm(a, y, g("ln2_g"), g("ln2_b"))
    up = oracle.linear(hh, g("w_up"), g("b_up"))
    gl = np.vectorize(lambda t: oracle.gelu(float(t)))(up).astype(np.float32)
    return a + oracle.linear(gl, g("w_down"), g("b_down")), qkv


def test_combination_is_explicit_sum_and_first_layer_identity():
    shape = small_shape(n_branch=3, n_layer=2)
    w = rand_weights(shape)
    ids = ki.uniform_tokens(9, shape.vocab, 1, shape.seqlen)[0].numpy()
    orc = oracle.Oracle(shape, wbits(w))
    _, lo = orc.prefill(ids, want_layer_out=True)
    x0 = (w["wte"].float()[torch.as_tensor(ids, dtype=torch.long)] + w["wpe"].float()[:len(ids)]).numpy()
    # layer 1: every sub-layer reads the shared embedding and y is that embedding, once
    for n in range(3):
        out, _ = sublayer_from_steps(shape, w, 0, n, x0, x0)
        assert np.max(np.abs(out - lo[0, n])) < 1e-5
    wrong, _ = sublayer_from_steps(shape, w, 0, 0, x0, 3 * x0)
    assert np.max(np.abs(wrong - lo[0, 0])) > 1e-3       # y = N * x0 is a different function
    wrong, _ = sublayer_from_steps(shape, w, 0, 0, x0, 0 * x0)
    assert np.max(np.abs(wrong - lo[0, 0])) > 1e-3       # and so is y = 0
    # layer 2: y is the explicit sum of the three separately computed layer-1 outputs
    y = lo[0, 0].astype(np.float64) + lo[0, 1] + lo[0, 2]
    for n in range(3):
        out, _ = sublayer_from_steps(shape, w, 1, n, lo[0, n], y.astype(np.float32))
        assert np.max(np.abs(out - lo[1, n])) < 1e-5
    wrong, _ = sublayer_from_steps(shape, w, 1, 0, lo[0, 0], (y / 3).astype(np.float32))
    assert np.max(np.abs(wrong - lo[1, 0])) > 1e-3       # a mean is not the paper's sum


def test_identical_branches_stay_identical():
    shape = small_shape(n_branch=4, n_layer=3)
    w = rand_weights(shape)
    for k, v in w.items():
        if v is not None and v.dim() >= 3 and v.shape[1] == 4:
            w[k] = v[:, :1].expand(-1, 4, *v.shape[2:]).contiguous()
    ids = ki.uniform_tokens(11, shape.vocab, 1, shape.seqlen)[0].numpy()
    _, lo = oracle.Oracle(shape, wbits(w)).prefill(ids, want_layer_out=True)
    for n in range(1, 4):
        assert np.array_equal(lo[:, 0], lo[:, n])
    # with equal streams y = N * x from the second layer on
    y = 4 * lo[0, 0]
    out, _ = sublayer_from_steps(shape, w, 1, 2, lo[0, 2], y)
    assert np.max(np.abs(out - lo[1, 2])) < 1e-5


def test_branch_permutation_invariance():
    shape = small_shape(n_branch=3, n_layer=3)
    w = rand_weights(shape)
    ids = ki.uniform_tokens(13, shape.vocab, 1, shape.seqlen)[0].numpy()
    ref, _ = oracle.Oracle(shape, wbits(w)).prefill(ids)
    perm = [2, 0, 1]
    d = shape.d_model
    wp = dict(w)
    for k, v in w.items():
        if v is not None and v.dim() >= 3 and v.shape[1] == 3:
            wp[k] = v[:, perm].contiguous()
    wp["w_concat"] = torch.cat([w["w_concat"][:, p * d:(p + 1) * d] for p in perm], dim=1).contiguous()
    got, _ = oracle.Oracle(shape, wbits(wp)).prefill(ids)
    assert np.max(np.abs(got - ref)) < 1e-5
    # permuting the branches without W_concat's column blocks must change the result
    wp["w_concat"] = w["w_concat"]
    bad, _ = oracle.Oracle(shape, wbits(wp)).prefill(ids)
    assert np.max(np.abs(bad - ref)) > 1e-3


def test_zeroed_residual_branches_closed_form():
    """With Wo, W2 and their biases zero every stream stays x0, so
    logits = LN_f(x0 . sum_n Wc[n]^T + bc) . wte^T."""
    shape = small_shape(n_branch=3, n_layer=2)
    w = rand_weights(shape)
    for k in ("w_proj", "b_proj", "w_down", "b_down"):
        w[k] = torch.zeros_like(w[k])
    ids = ki.uniform_tokens(17, shape.vocab, 1, shape.seqlen)[0].numpy()
    got, _ = oracle.Oracle(shape, wbits(w)).prefill(ids)
    d = shape.d_model
    W = {k: v.double().numpy() for k, v in w.items()}
    x0 = W["wte"][ids] + W["wpe"][:len(ids)]
    wc = sum(W["w_concat"][:, n * d:(n + 1) * d] for n in range(3))
    z = x0 @ wc.T + W["b_concat"]
    zn = (z - z.mean(1, keepdims=True)) / np.sqrt(z.var(1, keepdims=True) + 1e-5) * W["lnf_g"] + W["lnf_b"]
    ref = zn @ W["wte"].T
    assert np.max(np.abs(got - ref)) < 2e-5 * max(1.0, np.max(np.abs(ref)))


# ------------------------------------------------------------------ causality, cache, decode

def test_causality_bit_exact():
    shape = small_shape()
    w = rand_weights(shape)
    ids = ki.uniform_tokens(19, shape.vocab, 1, shape.seqlen)[0].numpy()
    ref, _ = oracle.Oracle(shape, wbits(w)).prefill(ids)
    t = 6
    ids2 = ids.copy()
    ids2[t + 1:] = (ids2[t + 1:] + 31) % shape.vocab
    got, _ = oracle.Oracle(shape, wbits(w)).prefill(ids2)
    assert np.array_equal(got[:t + 1], ref[:t + 1])
    assert not np.array_equal(got[t + 1:], ref[t + 1:])
    # a shorter prompt gives the same logits on its positions
    short, _ = oracle.Oracle(shape, wbits(w)).prefill(ids[:t + 1])
    assert np.array_equal(short, ref[:t + 1])


@pytest.mark.parametrize("bf16_store", [False, True])
def test_prefill_then_decode_equals_longer_prefill(bf16_store):
    shape = small_shape(seqlen=14)
    w = rand_weights(shape)
    ids = ki.uniform_tokens(23, shape.vocab, 1, 14)[0].numpy()
    full = oracle.Oracle(shape, wbits(w), bf16_store=bf16_store)
    ref, _ = full.prefill(ids)
    inc = oracle.Oracle(shape, wbits(w), bf16_store=bf16_store)
    first, _ = inc.prefill(ids[:9])
    assert np.max(np.abs(first - ref[:9])) < 1e-5
    for t in range(9, 14):
        step = inc.decode_step(int(ids[t]))
        assert np.max(np.abs(step - ref[t])) < 1e-5
    assert inc.cur_len == 14
    for layer in range(shape.n_layer):
        for n in range(shape.n_branch):
            for which in (0, 1):
                assert np.max(np.abs(inc.cache(layer, n, which) - full.cache(layer, n, which))) < 1e-5


def test_cache_holds_qkv_rows_by_head():
    shape = small_shape()
    w = rand_weights(shape)
    ids = ki.uniform_tokens(29, shape.vocab, 1, shape.seqlen)[0].numpy()
    orc = oracle.Oracle(shape, wbits(w))
    orc.prefill(ids)
    d, H = shape.d_model, shape.n_head
    hd = d // H
    x0 = (w["wte"].float()[torch.as_tensor(ids, dtype=torch.long)] + w["wpe"].float()[:len(ids)]).numpy()
    for n in range(shape.n_branch):
        _, qkv = sublayer_from_steps(shape, w, 0, n, x0, x0)
        for which in (0, 1):
            c = orc.cache(0, n, which)  # [H, l, hd]
            for h in range(H):
                lo = d * (1 + which) + h * hd
                assert np.max(np.abs(c[h] - qkv[:, lo:lo + hd])) < 1e-6


def test_bf16_store_mode_rounds_the_cache_and_stays_close():
    shape = ki.CONFIGS["C0"]
    w = ki.make_weights(shape, seed=0)
    ids = ki.uniform_tokens(1, shape.vocab, 1, 32)[0].numpy()
    a = oracle.Oracle(shape, wbits(w))
    b = oracle.Oracle(shape, wbits(w), bf16_store=True)
    la, _ = a.prefill(ids)
    lb, _ = b.prefill(ids)
    rel = np.linalg.norm(la - lb) / np.linalg.norm(la)
    assert 0 < rel < 1e-2
    kc = b.cache(1, 1, 0)
    assert np.array_equal(kc, torch.from_numpy(kc).to(torch.bfloat16).float().numpy())
    assert not np.array_equal(a.cache(1, 1, 0), kc)


def test_error_codes():
    shape = small_shape()
    w = rand_weights(shape)
    orc = oracle.Oracle(shape, wbits(w))
    with pytest.raises(RuntimeError, match="-3"):
        orc.prefill(np.array([1, 2, shape.vocab], dtype=np.int32))
    with pytest.raises(RuntimeError, match="-2"):
        orc.prefill(np.zeros(shape.max_pos + 1, dtype=np.int32))
    with pytest.raises(RuntimeError):
        orc.decode_step(0)  # nothing prefilled yet


# ------------------------------------------------------------------ configuration arithmetic

def test_parameter_counts_match_paper_tables():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "paper_param_tables.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 21
    for r in rows:
        kind = r[0]
        if kind == "table1":
            N, L, d, printed = int(r[1]), int(r[2]), int(r[3]), float(r[4])
            got = ki.param_count(N, L, d, 50257, 2 * d, max_pos=1024, with_concat=True) / 1e6
            assert abs(got - printed) / printed < 2e-3, (r, got)
        elif kind == "table3":
            N, d, printed = int(r[1]), int(r[2]), float(r[3])
            got = (ki.param_count(N, 1, d, 0, 2 * d)) / 1e6
            assert abs(got - printed) / printed < 3e-3, (r, got)
        else:
            d, printed = int(r[2]), float(r[3])
            got = ki.param_count(1, 1, d, 0, 4 * d) / 1e6
            assert abs(got - printed) / printed < 3e-3, (r, got)


def test_engine_configs_follow_table3():
    """The K* workloads are the Kraken columns of Table 3: (degree, width) pairs as printed, FFN 2 d, vocabulary
    51,200, 2048-token context, batch 1 (Sec. 4.2), and the TTFT table names only those workloads."""
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "paper_param_tables.txt"))
            if ln.strip() and not ln.startswith("#")]
    printed = {(int(r[1]), int(r[2])) for r in rows if r[0] == "table3"}
    engines = {k: s for k, s in ki.CONFIGS.items() if k.startswith("K") and not k.startswith("K0")}
    assert {(s.n_branch, s.d_model) for s in engines.values()} == printed
    for s in engines.values():
        assert s.d_ff == 2 * s.d_model and s.vocab == 51200 and s.max_pos == 2048 and s.batch == 1
        assert s.d_model % s.n_head == 0 and s.head_dim in (72, 96, 104, 128)
    assert set(ki.PAPER_TTFT_MS) == set(engines)
    assert all(set(v) == {128, 2048} for v in ki.PAPER_TTFT_MS.values())


# ------------------------------------------------------------------ grouped-query / multi-query attention

@pytest.mark.parametrize("n_head,n_kv", [(4, 2), (4, 1), (6, 3), (2, 2)])
def test_grouped_query_attention_equals_multi_head_with_repeated_kv(n_head, n_kv):
    """Grouped-query attention (the KV-cache mitigation named in Sec. 4.2) is multi-head attention whose
    key / value projections are shared by the query heads of a group: copying each shared K and V
    projection to every query head of its group gives a multi-head model with the same logits, and the
    grouped cache holds one row set per key/value head."""
    hd = 8
    d = n_head * hd
    g_shape = small_shape(d_model=d, n_head=n_head, d_ff=2 * d, n_kv_head=n_kv)
    m_shape = small_shape(d_model=d, n_head=n_head, d_ff=2 * d)
    wg = rand_weights(g_shape)
    assert wg["w_qkv"].shape[2] == d + 2 * n_kv * hd
    rep = n_head // n_kv
    kvd = n_kv * hd
    idx = torch.arange(n_head * hd)
    src = (idx // hd // rep) * hd + idx % hd                      # column of the shared head for each MHA column
    wm = dict(wg)
    wq, wk, wv = wg["w_qkv"][:, :, :d], wg["w_qkv"][:, :, d:d + kvd], wg["w_qkv"][:, :, d + kvd:]
    wm["w_qkv"] = torch.cat([wq, wk[:, :, src], wv[:, :, src]], dim=2).contiguous()
    bq, bk, bv = wg["b_qkv"][:, :, :d], wg["b_qkv"][:, :, d:d + kvd], wg["b_qkv"][:, :, d + kvd:]
    wm["b_qkv"] = torch.cat([bq, bk[:, :, src], bv[:, :, src]], dim=2).contiguous()
    ids = ki.uniform_tokens(9, g_shape.vocab, 1, g_shape.seqlen)[0].numpy()
    og, om = oracle.Oracle(g_shape, wbits(wg)), oracle.Oracle(m_shape, wbits(wm))
    lg, _ = og.prefill(ids[:-2])
    lm, _ = om.prefill(ids[:-2])
    assert np.array_equal(lg, lm)
    for t in ids[-2:]:                                            # and through decode steps
        assert np.array_equal(og.decode_step(int(t)), om.decode_step(int(t)))
    for layer in range(g_shape.n_layer):
        for which in (0, 1):
            cg, cm = og.cache(layer, 1, which), om.cache(layer, 1, which)
            assert cg.shape == (n_kv, len(ids), hd) and cm.shape == (n_head, len(ids), hd)
            for h in range(n_head):
                assert np.array_equal(cm[h], cg[h // rep])


def test_kv_heads_equal_to_heads_is_plain_multi_head():
    a, b = small_shape(), small_shape(n_kv_head=2)
    w = rand_weights(a)
    ids = ki.uniform_tokens(9, a.vocab, 1, a.seqlen)[0].numpy()
    la, _ = oracle.Oracle(a, wbits(w)).prefill(ids)
    lb, _ = oracle.Oracle(b, wbits(w)).prefill(ids)
    assert np.array_equal(la, lb)
    with pytest.raises(ValueError):
        oracle.Oracle(small_shape(n_kv_head=3), wbits(w))       # 2 heads cannot share 3 key/value heads


# ------------------------------------------------------------------ IEEE half as the 16-bit type

def test_half_rounding_and_widening_against_numpy():
    """The oracle's half conversions against numpy's float16 (an independent implementation): every bit
    pattern widens to the same value; rounding agrees on ties, subnormals, overflow and a random sweep."""
    pats = np.arange(65536, dtype=np.uint16)
    want = pats.view(np.float16).astype(np.float32)
    got = np.array([oracle.f16_to_f32(int(b)) for b in pats[::7]], dtype=np.float32)
    w = want[::7]
    assert np.array_equal(np.isnan(got), np.isnan(w))
    assert np.array_equal(got[~np.isnan(w)], w[~np.isnan(w)])
    cases = [1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 2049.0, 2051.0, 65504.0, 65519.9, 65520.0, 70000.0, -70000.0,
             6e-8, 5.96e-8, 2.98e-8, 2.9e-8, 1e-7, -1e-7, 6.1e-5, 0.1, -0.3333, 0.0]
    rng = np.random.default_rng(0)
    cases += list(rng.normal(0, 1, 2000).astype(np.float32)) + list(rng.normal(0, 1e-5, 500).astype(np.float32))
    for x in cases:
        with np.errstate(over="ignore"):
            ref = float(np.float32(x).astype(np.float16).astype(np.float32))
        assert oracle.round_f16(float(np.float32(x))) == ref, x


def test_half_mode_matches_library_composition_and_rounds_stores_to_half():
    shape = small_shape()
    w = {k: (None if v is None else v.to(torch.float16)) for k, v in rand_weights(shape).items()}
    ids = ki.uniform_tokens(7, shape.vocab, 1, shape.seqlen)[0].numpy()
    ref, _ = torch_kraken(shape, w, ids, final_ln=True)
    got, _ = oracle.Oracle(shape, wbits(w), half=True).prefill(ids)
    assert np.max(np.abs(got - ref)) < 2e-5 * max(1.0, np.max(np.abs(ref)))
    # the same patterns read as bfloat16 are a different model
    other, _ = oracle.Oracle(shape, wbits(w), half=False).prefill(ids)
    assert np.max(np.abs(other - ref)) > 1e-2
    # store points round to half: LayerNorm output
    a = np.random.default_rng(1).normal(0, 1, (5, 32)).astype(np.float32)
    g = bits(torch.ones(32, dtype=torch.float16))
    plain = oracle.layernorm(a, None, g, None, half=True)
    rounded = oracle.layernorm(a, None, g, None, round_out=True, half=True)
    assert np.array_equal(rounded, plain.astype(np.float16).astype(np.float32))
    # and the cache of a store-rounding run holds values exactly representable in half
    orc = oracle.Oracle(shape, wbits(w), bf16_store=True, half=True)
    orc.prefill(ids)
    k = orc.cache(0, 0, 0)
    assert np.array_equal(k, k.astype(np.float16).astype(np.float32))


# ------------------------------------------------------------------ comparison architectures of Sec. 4.2

def test_parallel_attention_feedforward_variant_is_a_gptj_style_stack():
    """parallel_ffn = 1 (with one branch and no cross-branch term): out = x + MHA(LN(x)) + FFN(LN(x)), one
    LayerNorm per layer, written here from library routines without any Kraken notion."""
    shape = small_shape(n_branch=1, n_layer=3, no_combine=1, parallel_ffn=1)
    w = rand_weights(shape)
    w["w_concat"] = torch.eye(shape.d_model, dtype=torch.bfloat16)
    w["b_concat"] = None
    ids = ki.uniform_tokens(5, shape.vocab, 1, shape.seqlen)[0].numpy()
    W = {k: (None if v is None else v.double()) for k, v in w.items()}
    d, H = shape.d_model, shape.n_head
    l = len(ids)
    x = W["wte"][torch.as_tensor(ids, dtype=torch.long)] + W["wpe"][:l]
    for layer in range(shape.n_layer):
        u = F.layer_norm(x, (d,), W["ln1_g"][layer, 0], W["ln1_b"][layer, 0], 1e-5)
        qkv = F.linear(u, W["w_qkv"][layer, 0], W["b_qkv"][layer, 0])
        q, k, v = [t.reshape(l, H, d // H).transpose(0, 1) for t in qkv.split(d, dim=1)]
        o = F.scaled_dot_product_attention(q[None], k[None], v[None], is_causal=True)[0].transpose(0, 1).reshape(l, d)
        attn = F.linear(o, W["w_proj"][layer, 0], W["b_proj"][layer, 0])
        ffn = F.linear(F.gelu(F.linear(u, W["w_up"][layer, 0], W["b_up"][layer, 0])),
                       W["w_down"][layer, 0], W["b_down"][layer, 0])
        x = x + attn + ffn
    ref = (F.layer_norm(x, (d,), W["lnf_g"], W["lnf_b"], 1e-5) @ W["wte"].T).numpy()
    got, _ = oracle.Oracle(shape, wbits(w)).prefill(ids)
    assert np.max(np.abs(got - ref)) < 2e-5 * max(1.0, np.max(np.abs(ref)))
    # it is a different function from the sequential stack on the same weights
    seq, _ = oracle.Oracle(small_shape(n_branch=1, n_layer=3, no_combine=1), wbits(w)).prefill(ids)
    assert np.max(np.abs(seq - ref)) > 1e-3



# ------------------------------------------------------------------ the store points of the rounding mode

STORE_POINTS = ("ln1", "qkv", "o", "ln2", "gelu", "concat_in", "zf")


def forward_with_explicit_rounding(shape, w, ids, half, final_ln, skip=None):
    """Algorithm 1 plus the tail, assembled from the individually pinned step functions, with a round-to-16-bit
    written out after each store point of a "16-bit activations, fp32 accumulate" implementation: the two
    LayerNorm outputs, q | k | v (hence the cache), the attention output, the GELU output, the rows that
    W_concat reads and the rows that the unembedding reads.  The residual stream (x0, a, x_n, y) is never
    rounded.  The rounding itself is numpy's / torch's conversion, not the oracle's.  `skip` leaves one
    store point unrounded (the negative controls)."""
    def rnd(name, x):
        if name == skip:
            return x
        x = np.ascontiguousarray(x, dtype=np.float32)
        if half:
            return x.astype(np.float16).astype(np.float32)
        return torch.from_numpy(x).to(torch.bfloat16).float().numpy()

    N, L, d, H = shape.n_branch, shape.n_layer, shape.d_model, shape.n_head
    hd = d // H
    n = len(ids)
    x0 = (w["wte"].float()[torch.as_tensor(ids, dtype=torch.long)] + w["wpe"].float()[:n]).numpy()
    x = [x0.copy() for _ in range(N)]
    layer_out = np.zeros((L, N, n, d), dtype=np.float32)
    caches = {}
    for l in range(L):
        y = x0 if l == 0 else np.sum(np.stack(x).astype(np.float64), axis=0).astype(np.float32)
        nxt = []
        for b in range(N):
            g = lambda k: bits(w[k][l, b])
            u = rnd("ln1", oracle.layernorm(x[b], None, g("ln1_g"), g("ln1_b"), half=half))
            qkv = rnd("qkv", oracle.linear(u, g("w_qkv"), g("b_qkv"), half=half))
            caches[(l, b, 0)] = qkv[:, d:2 * d].reshape(n, H, hd).transpose(1, 0, 2)
            caches[(l, b, 1)] = qkv[:, 2 * d:].reshape(n, H, hd).transpose(1, 0, 2)
            o = np.zeros((n, d), dtype=np.float32)
            for h in range(H):
                sl = slice(h * hd, (h + 1) * hd)
                o[:, sl] = oracle.attention_head(qkv[:, sl], qkv[:, d:2 * d][:, sl], qkv[:, 2 * d:][:, sl])
            o = rnd("o", o)
            a = x[b] + oracle.linear(o, g("w_proj"), g("b_proj"), half=half)
            hh = rnd("ln2", oracle.layernorm(a, y, g("ln2_g"), g("ln2_b"), half=half))
            up = oracle.linear(hh, g("w_up"), g("b_up"), half=half)
            gl = rnd("gelu", np.vectorize(lambda t: oracle.gelu(float(t)))(up).astype(np.float32))
            out = a + oracle.linear(gl, g("w_down"), g("b_down"), half=half)
            layer_out[l, b] = out
            nxt.append(out)
        x = nxt
    cat = rnd("concat_in", np.concatenate(x, axis=1))                        # branch-major
    z = oracle.linear(cat, bits(w["w_concat"]), bits(w["b_concat"]), half=half)
    if final_ln:
        zf = rnd("zf", oracle.layernorm(z, None, bits(w["lnf_g"]), bits(w["lnf_b"]), half=half))
    else:
        zf = rnd("zf", z)
    logits = oracle.linear(zf, bits(w["wte"]), None, half=half)
    return logits, layer_out, caches


@pytest.mark.parametrize("half", [False, True])
@pytest.mark.parametrize("final_ln", [True, False])
def test_rounding_mode_rounds_exactly_at_the_store_points(half, final_ln):
    """The mode that decides the arg-max criterion and the cache comparison: its sub-layer outputs, cache rows
    and logits equal, bit for bit, the composition above with every rounding written out; leaving any single
    rounding out gives different logits, so none of the store points is missing from (or extra in) the oracle."""
    shape = small_shape(n_branch=2, n_layer=2, seqlen=10)
    w = rand_weights(shape)
    if half:
        w = {k: (None if v is None else v.to(torch.float16)) for k, v in w.items()}
    ids = ki.uniform_tokens(13, shape.vocab, 1, shape.seqlen)[0].numpy()
    orc = oracle.Oracle(shape, wbits(w), bf16_store=True, half=half, final_ln=final_ln)
    got, lo = orc.prefill(ids, want_layer_out=True)
    want, want_lo, want_cache = forward_with_explicit_rounding(shape, w, ids, half, final_ln)
    assert np.array_equal(lo, want_lo)
    for (l, b, which), rows in want_cache.items():
        assert np.array_equal(orc.cache(l, b, which), rows), (l, b, which)
    assert np.array_equal(got, want)
    # the unrounded mode is a different function at every one of these outputs
    plain, plain_lo = oracle.Oracle(shape, wbits(w), half=half, final_ln=final_ln).prefill(ids, want_layer_out=True)
    assert not np.array_equal(plain, got) and not np.array_equal(plain_lo, lo)
    for point in STORE_POINTS:
        other, other_lo, _ = forward_with_explicit_rounding(shape, w, ids, half, final_ln, skip=point)
        assert not np.array_equal(other, got), point
        if point in ("concat_in", "zf"):
            assert np.array_equal(other_lo, lo), point           # the tail's roundings do not touch the layers
        else:
            assert not np.array_equal(other_lo, lo), point
