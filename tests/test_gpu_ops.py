"""Each CUDA kernel of the path, called through the C ABI, against the oracle's matching step."""
import ctypes as C

import numpy as np
import pytest
import torch

import kraken_inputs as ki
import oracle
import paper_2408_07802_b200 as kr

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def bits(t):
    return ki.bf16_tensor_to_bits(t)


def bf16_ulp_close(got: np.ndarray, ref: np.ndarray, ulps=1.0, atol=1e-6):
    """got (bf16 values as fp32) within `ulps` bf16 steps of ref (fp32)."""
    tol = ulps * np.abs(ref) * 2.0 ** -7 + atol
    bad = np.abs(got - ref) > tol
    return not bad.any(), float(np.max(np.abs(got - ref) - tol))


# ------------------------------------------------------------------ embedding

def test_embed_and_bad_token_flag():
    V, P, d = 300, 50, 128
    wte = ki.normal_bf16(1, 0, (V, d), 0.5, DEV)
    wpe = ki.normal_bf16(1, 1, (P, d), 0.5, DEV)
    ids = ki.uniform_tokens(2, V, 3, 17, DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = kr.op_embed(ids.reshape(-1), 17, 5, wte, wpe, status).cpu().numpy()
    pos = np.tile(np.arange(5, 22), 3)
    ref = wte.float().cpu().numpy()[ids.cpu().numpy().reshape(-1)] + wpe.float().cpu().numpy()[pos]
    assert np.array_equal(out, ref)
    assert int(status.item()) == 0
    bad = ids.clone().reshape(-1)
    bad[4] = V
    bad[9] = -1
    out2 = kr.op_embed(bad, 17, 5, wte, wpe, status).cpu().numpy()
    assert int(status.item()) & 1
    assert np.array_equal(out2[4], wte.float().cpu().numpy()[0] + wpe.float().cpu().numpy()[pos[4]])
    assert np.array_equal(out2[5], ref[5])


# ------------------------------------------------------------------ LayerNorm

@pytest.mark.parametrize("d", [128, 768, 2048, 2496, 4096, 7424])
@pytest.mark.parametrize("with_y", [False, True])
def test_layernorm(d, with_y):
    G, rows = 3, 37
    a = (ki.normal_bf16(3, 0, (G, rows, d), 1.0, DEV).float() * 1.7 + 0.3).contiguous()
    y = ki.normal_bf16(3, 1, (rows, d), 2.0, DEV).float().contiguous() if with_y else None
    gamma = (1 + ki.normal_bf16(3, 2, (G, d), 0.3, DEV).float()).to(torch.bfloat16)
    beta = ki.normal_bf16(3, 3, (G, d), 0.3, DEV)
    out = kr.op_layernorm(a, y, gamma, beta).float().cpu().numpy()
    for g in range(G):
        ref = oracle.layernorm(a[g].cpu().numpy(), None if y is None else y.cpu().numpy(), bits(gamma[g]),
                               bits(beta[g]))
        ok, worst = bf16_ulp_close(out[g], ref, ulps=1.0, atol=1e-5)
        assert ok, (g, worst)
    # one input shared by every group, no beta
    out2 = kr.op_layernorm(a[0].contiguous(), y, gamma, None, shared_a=True).float().cpu().numpy()
    ref = oracle.layernorm(a[0].cpu().numpy(), None if y is None else y.cpu().numpy(), bits(gamma[2]), None)
    ok, worst = bf16_ulp_close(out2[2], ref, ulps=1.0, atol=1e-5)
    assert ok, worst


@pytest.mark.parametrize("G,d,with_y", [(4, 2048, True), (4, 2048, False), (2, 768, True), (1, 1000, False),
                                        (3, 512, True), (8, 512, True), (8, 1920, True), (5, 768, True), (16, 256, False),
                                        (4, 2496, True), (4, 3120, False), (2, 4096, True)])
def test_layernorm_many_rows_persistent_kernel(G, d, with_y):
    """With a status word and many rows the persistent ring kernel runs: sampled rows against the oracle,
    every row bit-equal to the warp-per-row kernel (same operations in the same order); ragged row count."""
    rows = 8 * torch.cuda.get_device_properties(0).multi_processor_count + 37
    a = (ki.normal_bf16(4, 0, (G, rows, d), 1.0, DEV).float() * 1.3 - 0.2).contiguous()
    y = ki.normal_bf16(4, 1, (rows, d), 2.0, DEV).float().contiguous() if with_y else None
    gamma = (1 + ki.normal_bf16(4, 2, (G, d), 0.3, DEV).float()).to(torch.bfloat16)
    beta = ki.normal_bf16(4, 3, (G, d), 0.3, DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = kr.op_layernorm(a, y, gamma, beta, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    with kr.tuning(kr.TUNE_LN_ROW_KERNEL, 1):          # the warp-per-row kernel, not one CTA per row
        plain = kr.op_layernorm(a, y, gamma, beta)
    assert torch.equal(out.view(torch.int16), plain.view(torch.int16))
    pick = [0, 1, rows // 2, rows - 38, rows - 1]
    for g in (0, G - 1):
        ref = oracle.layernorm(a[g][pick].cpu().numpy(), None if y is None else y[pick].cpu().numpy(),
                               bits(gamma[g]), bits(beta[g]))
        ok, worst = bf16_ulp_close(out[g][pick].float().cpu().numpy(), ref, ulps=1.0, atol=1e-5)
        assert ok, (g, worst)


@pytest.fixture(autouse=True)
def _library_choices_restored():
    """Every test starts and ends with the library's own kernel choices."""
    yield
    for key in (kr.TUNE_LN_ROW_KERNEL, kr.TUNE_ATTN_SCHEDULE):
        kr.set_tuning(key, 0)


@pytest.mark.parametrize("force", [1, 2])
def test_layernorm_one_cta_per_row_walks_many_rows(force):
    """Rows wider than 4096 take the one-CTA-per-row kernel, whose grid is smaller than the number of rows here, so
    every CTA walks several rows; the same call forced onto the warp-per-row kernel agrees within one bf16 step
    (the two sum in different orders)."""
    kr.set_tuning(kr.TUNE_LN_ROW_KERNEL, force)      # 1: one warp per row, 2: one CTA per row
    G, d = 2, 4992
    rows = 5 * torch.cuda.get_device_properties(0).multi_processor_count + 3
    a = (ki.normal_bf16(5, 0, (G, rows, d), 1.0, DEV).float() * 0.9 + 0.1).contiguous()
    y = ki.normal_bf16(5, 1, (rows, d), 2.0, DEV).float().contiguous()
    gamma = (1 + ki.normal_bf16(5, 2, (G, d), 0.3, DEV).float()).to(torch.bfloat16)
    beta = ki.normal_bf16(5, 3, (G, d), 0.3, DEV)
    out = kr.op_layernorm(a, y, gamma, beta)
    pick = [0, 1, rows // 3, rows - 2, rows - 1]
    for g in range(G):
        ref = oracle.layernorm(a[g][pick].cpu().numpy(), y[pick].cpu().numpy(), bits(gamma[g]), bits(beta[g]))
        ok, worst = bf16_ulp_close(out[g][pick].float().cpu().numpy(), ref, ulps=1.0, atol=1e-5)
        assert ok, (g, worst)


# ------------------------------------------------------------------ grouped GEMM

def gemm_case(G, M, Nout, K, epi, n_tile, seed=0, integer=False, shared_resid=False, w_constant=0):
    if integer:
        a = (ki.hash32(seed, 60, 0, G * M * K, DEV) % 5 - 2).to(torch.bfloat16).reshape(G, M, K)
        w = (ki.hash32(seed, 61, 0, G * Nout * K, DEV) % 5 - 2).to(torch.bfloat16).reshape(G, Nout, K)
        bias = (ki.hash32(seed, 62, 0, G * Nout, DEV) % 7 - 3).to(torch.bfloat16).reshape(G, Nout)
    else:
        a = ki.normal_bf16(seed, 60, (G, M, K), 1.0, DEV)
        w = ki.normal_bf16(seed, 61, (G, Nout, K), 1.0 / np.sqrt(K), DEV)
        bias = ki.normal_bf16(seed, 62, (G, Nout), 0.5, DEV)
    args = kr.GemmArgs()
    args.a, args.a_gstride, args.lda = a.data_ptr(), M * K, K
    args.w, args.w_gstride, args.ldw = w.data_ptr(), Nout * K, K
    args.bias, args.bias_gstride = bias.data_ptr(), Nout
    args.groups, args.m, args.n_out, args.k = G, M, Nout, K
    args.epilogue, args.n_tile = epi, n_tile
    args.w_constant = w_constant
    keep = [a, w, bias]
    out_f32 = out_bf16 = resid = ssum = None
    if epi in (kr.EPI_F32, kr.EPI_RESID_F32, kr.EPI_RESID_SUM):
        out_f32 = torch.full((G, M, Nout), float("nan"), dtype=torch.float32, device=DEV)
        args.out_f32, args.out_f32_gstride, args.ld_out_f32 = out_f32.data_ptr(), M * Nout, Nout
    if epi in (kr.EPI_BF16, kr.EPI_GELU_BF16):
        out_bf16 = torch.full((G, M, Nout), float("nan"), dtype=torch.bfloat16, device=DEV)
        args.out_bf16, args.out_bf16_gstride, args.ld_out_bf16 = out_bf16.data_ptr(), M * Nout, Nout
    if epi in (kr.EPI_RESID_F32, kr.EPI_RESID_SUM):
        if integer:
            resid = (ki.hash32(seed, 63, 0, G * M * Nout, DEV) % 9 - 4).float().reshape(G, M, Nout)
        else:
            resid = ki.normal_bf16(seed, 63, (G, M, Nout), 1.0, DEV).float() * 1.37
        if shared_resid:
            resid = resid[:1].contiguous()
        args.resid, args.resid_gstride, args.ld_resid = resid.data_ptr(), 0 if shared_resid else M * Nout, Nout
    if epi == kr.EPI_RESID_SUM:
        ssum = torch.full((M, Nout), float("nan"), dtype=torch.float32, device=DEV)
        args.sum, args.ld_sum = ssum.data_ptr(), Nout
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    kr.op_grouped_gemm(args, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0

    # oracle
    ref = np.stack([oracle.linear(a[g].float().cpu().numpy(), bits(w[g]), bits(bias[g])) for g in range(G)])
    if resid is not None:
        r = resid.cpu().numpy()
        ref = ref + (r if not shared_resid else np.broadcast_to(r, ref.shape))
    if epi == kr.EPI_GELU_BF16:
        ref = np.vectorize(lambda t: oracle.gelu(float(t)))(ref).astype(np.float32)
    return dict(out_f32=None if out_f32 is None else out_f32.cpu().numpy(),
                out_bf16=None if out_bf16 is None else out_bf16.float().cpu().numpy(),
                sum=None if ssum is None else ssum.cpu().numpy(), ref=ref, keep=keep)


@pytest.mark.parametrize("n_tile", [32, 64, 96, 128, 160, 192, 224, 256, 512])
def test_gemm_integer_exact_ragged(n_tile):
    """Small integers make every product and partial sum exact: any mis-placed element shows."""
    r = gemm_case(2, 300, 200, 136, kr.EPI_F32, n_tile, integer=True)
    assert np.array_equal(r["out_f32"], r["ref"])


@pytest.mark.parametrize("n_tile", [64, 160, 512])
@pytest.mark.parametrize("Nout", [203, 330])
def test_gemm_bias_rows_not_aligned(n_tile, Nout):
    """An odd output width: the second group's bias row starts at an odd element, the last chunk of a tile is ragged
    (the epilogue warps park their bias values in shared memory piecewise then)."""
    r = gemm_case(2, 300, Nout, 136, kr.EPI_F32, n_tile, integer=True)
    assert np.array_equal(r["out_f32"], r["ref"])


@pytest.mark.parametrize("n_tile", [64, 256, 512])
@pytest.mark.parametrize("K", [136, 1000])
def test_gemm_constant_weights_fetched_before_the_predecessor_ends(n_tile, K):
    """w_constant: the first stages' W tiles are requested before the kernel waits for the stream's previous kernel
    (fewer k-blocks than stages, and more); several items per CTA, ragged edges; exact on small integers."""
    r = gemm_case(3, 700, 1100, K, kr.EPI_F32, n_tile, integer=True, w_constant=1)
    assert np.array_equal(r["out_f32"], r["ref"])


@pytest.mark.parametrize("n_tile", [0, 32, 64, 96, 128, 160, 192, 224, 256, 512])
def test_gemm_f32_many_tiles(n_tile):
    r = gemm_case(2, 2048, 2304, 768, kr.EPI_F32, n_tile, seed=1)
    err = np.abs(r["out_f32"] - r["ref"])
    assert err.max() < 2e-4, err.max()


@pytest.mark.parametrize("n_tile", [0, 96, 160, 512])
@pytest.mark.parametrize("epi", [kr.EPI_BF16, kr.EPI_GELU_BF16])
def test_gemm_bf16_epilogues(epi, n_tile):
    r = gemm_case(3, 200, 320, 256, epi, n_tile, seed=2)
    ok, worst = bf16_ulp_close(r["out_bf16"], r["ref"], ulps=1.0, atol=2e-4)
    assert ok, worst


@pytest.mark.parametrize("shared", [False, True])
def test_gemm_residual(shared):
    r = gemm_case(3, 260, 192, 320, kr.EPI_RESID_F32, 0, seed=3, shared_resid=shared)
    assert np.abs(r["out_f32"] - r["ref"]).max() < 2e-4


@pytest.mark.parametrize("n_tile", [64, 128, 512])
def test_gemm_cross_branch_sum(n_tile):
    """The AllReduce of Algorithm 1 inside the epilogue: sum equals the explicit sum of the branch outputs."""
    r = gemm_case(4, 700, 384, 512, kr.EPI_RESID_SUM, n_tile, seed=4)
    assert np.abs(r["out_f32"] - r["ref"]).max() < 3e-4
    explicit = r["ref"].astype(np.float64).sum(0)
    assert np.abs(r["sum"] - explicit).max() < 1e-3
    # integer case: bit exact, and equal to the sum of the kernel's own branch outputs in order
    r = gemm_case(4, 300, 256, 128, kr.EPI_RESID_SUM, n_tile, seed=5, integer=True)
    assert np.array_equal(r["out_f32"], r["ref"])
    assert np.array_equal(r["sum"], r["ref"].sum(0))


@pytest.mark.parametrize("hd,H,Hkv", [(64, 2, 2), (128, 1, 1), (104, 3, 3), (72, 2, 2), (96, 1, 1), (96, 3, 3),
                                       (64, 4, 2), (64, 4, 1), (104, 4, 2), (128, 2, 1)])
def test_gemm_qkv_scatter_is_index_exact(hd, H, Hkv):
    """One-hot activations times integer-coded weights: every cache element names its source.  Head dims that
    are not multiples of 32 (and widths that are not) take the path that stores 16-byte pieces."""
    d = H * hd
    G, batch, seqlen, pos0, P, K = 2, 3, 50, 7, 64, 64
    M = batch * seqlen
    t = torch.arange(M, device=DEV)
    a = torch.zeros(G, M, K, dtype=torch.bfloat16, device=DEV)
    a[:, t, t % K] = 1.0
    kvd = Hkv * hd                                                  # width of the K part and of the V part
    nout = d + 2 * kvd
    o = torch.arange(nout, device=DEV)[:, None]
    k = torch.arange(K, device=DEV)[None, :]
    w = torch.stack([((o * 7 + k * 13 + g * 29) % 251 - 125) for g in range(G)]).to(torch.bfloat16).contiguous()
    qbuf = torch.zeros(G, M, d, dtype=torch.bfloat16, device=DEV)
    cache = torch.full((G, 2, batch, Hkv, P, hd), -7.0, dtype=torch.bfloat16, device=DEV)
    args = kr.GemmArgs()
    args.a, args.a_gstride, args.lda = a.data_ptr(), M * K, K
    args.w, args.w_gstride, args.ldw = w.data_ptr(), nout * K, K
    args.groups, args.m, args.n_out, args.k = G, M, nout, K
    args.epilogue = kr.EPI_QKV
    args.n_kv_head = Hkv if Hkv != H else 0
    args.out_bf16, args.out_bf16_gstride, args.ld_out_bf16 = qbuf.data_ptr(), M * d, d
    args.k_cache, args.v_cache = cache[0, 0].data_ptr(), cache[0, 1].data_ptr()
    args.cache_gstride = cache.stride(0)
    args.seqlen, args.pos0, args.n_head, args.head_dim, args.max_pos = seqlen, pos0, H, hd, P
    kr.op_grouped_gemm(args)
    torch.cuda.synchronize()
    wf = w.float().cpu().numpy()
    got_q, got_c = qbuf.float().cpu().numpy(), cache.float().cpu().numpy()
    tk = np.arange(M) % K
    for g in range(G):
        assert np.array_equal(got_q[g], wf[g][:d, tk].T)
        for which in (0, 1):
            for b in range(batch):
                for h in range(Hkv):
                    rows = wf[g][d + which * kvd + h * hd: d + which * kvd + (h + 1) * hd]    # [hd, K]
                    want = rows[:, tk[b * seqlen:(b + 1) * seqlen]].T                          # [seqlen, hd]
                    assert np.array_equal(got_c[g, which, b, h, pos0:pos0 + seqlen], want)
                    # rows outside the written range are untouched
                    assert np.all(got_c[g, which, b, h, :pos0] == -7.0)
                    assert np.all(got_c[g, which, b, h, pos0 + seqlen:] == -7.0)


@pytest.mark.parametrize("G,M,Nout,K,epi,n_tile,with_y", [
    (2, 300, 768, 256, "resid", 64, True),        # twelve N tiles per row block, ragged last M tile
    (3, 700, 1024, 128, "sum", 512, False),       # CTA pairs, cross-branch sum and LayerNorm in one epilogue
    (1, 129, 520, 64, "resid", 256, True),        # ragged last N tile (8 columns), one row in the second M tile
    (2, 64, 96, 64, "resid", 32, False),          # one 32-column chunk per tile: half of the epilogue warps hold nothing
    (2, 512, 768, 192, "sum", 0, True),           # the library's own tile choice
    (4, 1024, 512, 64, "resid", 32, True),        # 512 tiles on 148 CTAs: row blocks straddle the rounds
    (4, 4096, 1024, 64, "sum", 512, False),       # 256 pair tiles on 74 pairs: the same for CTA pairs and the sum
])
def test_gemm_with_layernorm_behind_the_epilogue(G, M, Nout, K, epi, n_tile, with_y):
    """x = LN(out + y) in the kernel that produces `out` (Algorithm 1's two LayerNorm lines): the fp32 output and
    the cross-branch sum equal the oracle's linear step as without the LayerNorm, and the 16-bit LayerNorm output
    is within one bf16 step of the oracle's LayerNorm of those very rows.  Two launches in a row share the scratch."""
    kind = kr.EPI_RESID_F32 if epi == "resid" else kr.EPI_RESID_SUM
    a = ki.normal_bf16(5, 60, (G, M, K), 1.0, DEV)
    w = ki.normal_bf16(5, 61, (G, Nout, K), 1.0 / np.sqrt(K), DEV)
    bias = ki.normal_bf16(5, 62, (G, Nout), 0.5, DEV)
    resid = (ki.normal_bf16(5, 63, (G, M, Nout), 1.0, DEV).float() * 1.37 + 0.4).contiguous()
    y = (ki.normal_bf16(5, 64, (M, Nout), 2.0, DEV).float() - 0.7).contiguous() if with_y else None
    gamma = (1 + ki.normal_bf16(5, 65, (G, Nout), 0.3, DEV).float()).to(torch.bfloat16)
    beta = ki.normal_bf16(5, 66, (G, Nout), 0.3, DEV)
    args = kr.GemmArgs()
    args.a, args.a_gstride, args.lda = a.data_ptr(), M * K, K
    args.w, args.w_gstride, args.ldw = w.data_ptr(), Nout * K, K
    args.bias, args.bias_gstride = bias.data_ptr(), Nout
    args.groups, args.m, args.n_out, args.k = G, M, Nout, K
    args.epilogue, args.n_tile = kind, n_tile
    args.resid, args.resid_gstride, args.ld_resid = resid.data_ptr(), M * Nout, Nout
    nbytes = kr.gemm_ln_scratch_bytes(G, M, Nout, K, n_tile)
    scratch = torch.zeros(nbytes, dtype=torch.uint8, device=DEV)       # zeroed once, shared by both launches
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    for rep in range(2):
        out = torch.full((G, M, Nout), float("nan"), dtype=torch.float32, device=DEV)
        ssum = torch.full((M, Nout), float("nan"), dtype=torch.float32, device=DEV)
        ln_out = torch.full((G, M, Nout), float("nan"), dtype=torch.bfloat16, device=DEV)
        args.out_f32, args.out_f32_gstride, args.ld_out_f32 = out.data_ptr(), M * Nout, Nout
        if kind == kr.EPI_RESID_SUM:
            args.sum, args.ld_sum = ssum.data_ptr(), Nout
        ln = kr.GemmLnArgs()
        ln.ln_out, ln.ln_out_gstride, ln.ld_ln_out = ln_out.data_ptr(), M * Nout, Nout
        ln.gamma, ln.beta, ln.gb_gstride = gamma.data_ptr(), beta.data_ptr() if rep == 0 else None, Nout
        ln.y, ln.ld_y = (y.data_ptr() if with_y else None), Nout
        ln.eps = 1e-5
        ln.d_scratch, ln.scratch_bytes = scratch.data_ptr(), nbytes
        kr.op_grouped_gemm_ln(args, ln, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert int(scratch[:G * ((M + 255) // 256) * 8 * 8].view(torch.int32).abs().sum().item()) == 0   # counters back at zero
        got = out.cpu().numpy()
        for g in ([0, G - 1] if rep == 0 else [G // 2]):
            ref = oracle.linear(a[g].float().cpu().numpy(), bits(w[g]), bits(bias[g])) + resid[g].cpu().numpy()
            assert np.abs(got[g] - ref).max() < 3e-4, (g, np.abs(got[g] - ref).max())
            want = oracle.layernorm(got[g], y.cpu().numpy() if with_y else None, bits(gamma[g]),
                                    bits(beta[g]) if rep == 0 else None)
            ok, worst = bf16_ulp_close(ln_out[g].float().cpu().numpy(), want, ulps=1.0, atol=1e-5)
            assert ok, (rep, g, worst)
        if kind == kr.EPI_RESID_SUM:
            assert np.abs(ssum.cpu().numpy() - got.astype(np.float64).sum(0)).max() < 1e-4 * G


def test_gemm_with_layernorm_rejects_other_epilogues_and_small_scratch():
    G, M, Nout, K = 1, 64, 64, 64
    a = torch.zeros(G, M, K, dtype=torch.bfloat16, device=DEV)
    w = torch.zeros(G, Nout, K, dtype=torch.bfloat16, device=DEV)
    out = torch.zeros(G, M, Nout, dtype=torch.float32, device=DEV)
    lo = torch.zeros(G, M, Nout, dtype=torch.bfloat16, device=DEV)
    gamma = torch.ones(G, Nout, dtype=torch.bfloat16, device=DEV)
    args = kr.GemmArgs()
    args.a, args.a_gstride, args.lda = a.data_ptr(), M * K, K
    args.w, args.w_gstride, args.ldw = w.data_ptr(), Nout * K, K
    args.groups, args.m, args.n_out, args.k = G, M, Nout, K
    args.out_f32, args.out_f32_gstride, args.ld_out_f32 = out.data_ptr(), M * Nout, Nout
    args.resid, args.resid_gstride, args.ld_resid = out.data_ptr(), M * Nout, Nout
    args.n_tile = 64
    nbytes = kr.gemm_ln_scratch_bytes(G, M, Nout, K, 64)
    scratch = torch.zeros(nbytes, dtype=torch.uint8, device=DEV)
    ln = kr.GemmLnArgs()
    ln.ln_out, ln.ln_out_gstride, ln.ld_ln_out = lo.data_ptr(), M * Nout, Nout
    ln.gamma, ln.gb_gstride, ln.eps = gamma.data_ptr(), Nout, 1e-5
    ln.d_scratch, ln.scratch_bytes = scratch.data_ptr(), nbytes
    args.epilogue = kr.EPI_F32
    with pytest.raises(kr.KrakenError) as e:
        kr.op_grouped_gemm_ln(args, ln)
    assert e.value.status == kr.EINVAL
    args.epilogue = kr.EPI_RESID_F32
    ln.scratch_bytes = nbytes - 16
    with pytest.raises(kr.KrakenError) as e:
        kr.op_grouped_gemm_ln(args, ln)
    assert e.value.status == kr.ECAPACITY
    ln.scratch_bytes = nbytes
    kr.op_grouped_gemm_ln(args, ln)
    torch.cuda.synchronize()


def test_gemm_rejects_unaligned():
    a = torch.zeros(1, 8, 68, dtype=torch.bfloat16, device=DEV)
    args = kr.GemmArgs()
    args.a, args.lda, args.w, args.ldw = a.data_ptr(), 68, a.data_ptr(), 68
    args.groups, args.m, args.n_out, args.k = 1, 8, 8, 68
    args.epilogue = kr.EPI_F32
    out = torch.zeros(8, 8, device=DEV)
    args.out_f32, args.ld_out_f32 = out.data_ptr(), 8
    with pytest.raises(kr.KrakenError) as e:
        kr.op_grouped_gemm(args)
    assert e.value.status == kr.EUNSUPPORTED


# ------------------------------------------------------------------ attention

@pytest.mark.parametrize("hd", [64, 128, 72, 96, 104])
@pytest.mark.parametrize("seqlen,pos0", [(200, 0), (100, 37), (1, 90), (64, 0), (300, 0), (129, 127)])
def test_attention_matches_oracle(hd, seqlen, pos0):
    G, B, H, P = 2, 2, 2, 512
    d = H * hd
    q = ki.normal_bf16(7, 0, (G, B * seqlen, d), 1.0, DEV)
    kc = ki.normal_bf16(7, 1, (G, B, H, P, hd), 1.0, DEV)
    vc = ki.normal_bf16(7, 2, (G, B, H, P, hd), 1.0, DEV)
    # rows past the sequence hold garbage that must not leak (NaN would poison a masked product)
    kc[:, :, :, pos0 + seqlen:] = float("nan")
    vc[:, :, :, pos0 + seqlen:] = float("nan")
    out = kr.op_attention(q, kc, vc, B, seqlen, pos0, H).float().cpu().numpy()
    assert not np.isnan(out).any()
    qn, kn, vn = q.float().cpu().numpy(), kc.float().cpu().numpy(), vc.float().cpu().numpy()
    worst, num, den = 0.0, 0.0, 0.0
    for g in range(G):
        for b in range(B):
            for h in range(H):
                ref = oracle.attention_head(qn[g, b * seqlen:(b + 1) * seqlen, h * hd:(h + 1) * hd],
                                            kn[g, b, h, :pos0 + seqlen], vn[g, b, h, :pos0 + seqlen], q_pos0=pos0)
                got = out[g, b * seqlen:(b + 1) * seqlen, h * hd:(h + 1) * hd]
                worst = max(worst, np.abs(got - ref).max())
                num += ((got - ref) ** 2).sum()
                den += (ref ** 2).sum()
    assert worst < 3e-2, worst
    assert np.sqrt(num / den) < 6e-3, np.sqrt(num / den)


def test_attention_refuses_a_cache_with_gaps():
    """One kernel serves prefill attention; a cache whose sequences are further apart than heads x max_pos x
    head_dim (a view into a larger buffer) is refused with EUNSUPPORTED, not handed to a second kernel."""
    G, B, H, P, hd, seqlen = 1, 2, 2, 128, 64, 40
    q = ki.normal_bf16(9, 0, (G, B * seqlen, H * hd), 1.0, DEV)
    big = ki.normal_bf16(9, 1, (G, B, H + 1, P, hd), 1.0, DEV)
    kc = big[:, :, :H]                                       # sequences H + 1 heads apart
    with pytest.raises(kr.KrakenError) as e:
        kr.op_attention(q, kc, kc, B, seqlen, 0, H)
    assert e.value.status == kr.EUNSUPPORTED


def test_bounded_wait_runs_out_and_the_context_stays_usable():
    """Every device-side wait of the library has a limit; when it runs out the kernel leaves its loop, raises
    bit 1 of the status word and returns.  The probe waits, with that same routine, on a barrier that nothing
    signals: the status bit must appear, the kernel must return (no hang, no fault), and ordinary work on the
    same context afterwards must be correct."""
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    kr.test_wait_limit(status, 3000)                         # 3 ms
    t1.record()
    torch.cuda.synchronize()
    assert int(status.item()) == kr.STATUS_WAIT_LIMIT
    ms = t0.elapsed_time(t1)
    assert 2.0 <= ms <= 500.0, ms                            # it really waited, and it really stopped
    with pytest.raises(kr.KrakenError):
        kr.test_wait_limit(status, 0)
    # the context is intact: a LayerNorm launch right after gives the oracle's result
    a = ki.normal_bf16(31, 0, (1, 64, 256), 1.0, DEV).float().contiguous()
    gamma = (1 + ki.normal_bf16(31, 1, (1, 256), 0.3, DEV).float()).to(torch.bfloat16)
    out = kr.op_layernorm(a, None, gamma, None)
    ref = oracle.layernorm(a[0].cpu().numpy(), None, bits(gamma[0]), None)
    ok, worst = bf16_ulp_close(out[0].float().cpu().numpy(), ref, ulps=1.0, atol=1e-5)
    assert ok, worst


def test_tensor_core_issue_rate_one_and_two_issuing_threads():
    """The probe behind the attention kernel's roofline argument: 128 x 128 x 16 products issued by one thread
    cost clearly more than their 64 tensor cycles, 128 x 256 x 16 products run at the tensor rate (128), and two
    issuing threads in different warps reach the tensor rate with the small products too."""
    one = {f: kr.mma_issue_rate(f, 1) for f in range(7)}
    two = {f: kr.mma_issue_rate(f, 2) for f in (0, 1, 2, 3)}
    print("[probe] cycles per product, one issuing thread:", {k: round(v, 1) for k, v in one.items()},
          "two issuing threads:", {k: round(v, 1) for k, v in two.items()})
    assert 126 <= one[6] <= 134
    assert all(72 <= one[f] <= 130 for f in (0, 1, 2, 3, 4, 5)), one
    assert all(62 <= two[f] <= 70 for f in two), two


@pytest.mark.parametrize("G,B,H,hd,seqlen", [(4, 1, 16, 64, 768),     # one round of couples, a middle pair alone
                                              (4, 1, 16, 64, 1024),    # one round, every pair has a partner
                                              (4, 2, 16, 64, 1300),    # several rounds, ragged last tile
                                              (3, 2, 12, 128, 520)])   # fewer couples than SMs, ragged
def test_attention_fixed_work_lists_match_one_cta_per_item(G, B, H, hd, seqlen):
    """With more work items than SMs the kernel walks per-CTA lists of couples of items; each item's arithmetic
    is the same as with one CTA per item, so the outputs are equal bit for bit, and sampled heads match the
    oracle."""
    d = H * hd
    q = ki.normal_bf16(17, 0, (G, B * seqlen, d), 1.0, DEV)
    kc = ki.normal_bf16(17, 1, (G, B, H, seqlen, hd), 1.0, DEV)
    vc = ki.normal_bf16(17, 2, (G, B, H, seqlen, hd), 1.0, DEV)
    got = kr.op_attention(q, kc, vc, B, seqlen, 0, H)
    with kr.tuning(kr.TUNE_ATTN_SCHEDULE, 1):
        plain = kr.op_attention(q, kc, vc, B, seqlen, 0, H)
    torch.cuda.synchronize()
    assert torch.equal(got, plain)
    out = got.float().cpu().numpy()
    qn, kn, vn = q.float().cpu().numpy(), kc.float().cpu().numpy(), vc.float().cpu().numpy()
    for g, b, h in [(0, 0, 0), (G - 1, B - 1, H - 1), (1, 0, H // 2)]:
        ref = oracle.attention_head(qn[g, b * seqlen:(b + 1) * seqlen, h * hd:(h + 1) * hd], kn[g, b, h], vn[g, b, h])
        err = np.abs(out[g, b * seqlen:(b + 1) * seqlen, h * hd:(h + 1) * hd] - ref)
        assert err.max() < 3e-2, (g, b, h, err.max())


@pytest.mark.parametrize("hd,H,Hkv", [(64, 4, 2), (64, 8, 1), (128, 4, 1), (96, 6, 2), (64, 6, 2), (128, 2, 2)])
@pytest.mark.parametrize("seqlen,pos0", [(300, 0), (100, 37)])
def test_grouped_query_attention_matches_oracle(hd, H, Hkv, seqlen, pos0):
    """Query head h attends over key/value head h / (H / Hkv) (prefill kernel), against the oracle's
    single-head attention on the corresponding cache rows."""
    G, B, P = 2, 2, 512
    d = H * hd
    q = ki.normal_bf16(17, 0, (G, B * seqlen, d), 1.0, DEV)
    kc = ki.normal_bf16(17, 1, (G, B, Hkv, P, hd), 1.0, DEV)
    vc = ki.normal_bf16(17, 2, (G, B, Hkv, P, hd), 1.0, DEV)
    kc[:, :, :, pos0 + seqlen:] = float("nan")
    vc[:, :, :, pos0 + seqlen:] = float("nan")
    out = kr.op_attention(q, kc, vc, B, seqlen, pos0, H).float().cpu().numpy()
    assert not np.isnan(out).any()
    qn, kn, vn = q.float().cpu().numpy(), kc.float().cpu().numpy(), vc.float().cpu().numpy()
    worst = 0.0
    for g in range(G):
        for b in range(B):
            for h in range(H):
                hk = h // (H // Hkv)
                ref = oracle.attention_head(qn[g, b * seqlen:(b + 1) * seqlen, h * hd:(h + 1) * hd],
                                            kn[g, b, hk, :pos0 + seqlen], vn[g, b, hk, :pos0 + seqlen], q_pos0=pos0)
                worst = max(worst, np.abs(out[g, b * seqlen:(b + 1) * seqlen, h * hd:(h + 1) * hd] - ref).max())
    assert worst < 3e-2, worst


@pytest.mark.parametrize("hd,H,Hkv", [(64, 4, 2), (64, 8, 1), (128, 4, 1), (96, 6, 2), (64, 6, 2), (128, 16, 4)])
@pytest.mark.parametrize("n_keys,splits", [(1, 1), (131, 3), (700, 0), (2049, 32)])
def test_grouped_query_decode_attention_matches_oracle(hd, H, Hkv, n_keys, splits):
    """Decode step with shared key/value heads: the query heads of a group are served by one CTA (4, 2 or
    1 of them at a time)."""
    G, B, P = 2, 3, 2112
    d = H * hd
    q = ki.normal_bf16(18, 0, (G, B, d), 1.0, DEV)
    kc = ki.normal_bf16(18, 1, (G, B, Hkv, P, hd), 1.0, DEV)
    vc = ki.normal_bf16(18, 2, (G, B, Hkv, P, hd), 1.0, DEV)
    kc[:, :, :, n_keys:] = float("nan")
    vc[:, :, :, n_keys:] = float("nan")
    out = kr.op_decode_attention(q, kc, vc, n_keys, splits).float().cpu().numpy()
    assert not np.isnan(out).any()
    qn, kn, vn = q.float().cpu().numpy(), kc.float().cpu().numpy(), vc.float().cpu().numpy()
    worst = 0.0
    for g in range(G):
        for b in range(B):
            for h in range(H):
                hk = h // (H // Hkv)
                ref = oracle.attention_head(qn[g, b:b + 1, h * hd:(h + 1) * hd], kn[g, b, hk, :n_keys],
                                            vn[g, b, hk, :n_keys], q_pos0=n_keys - 1)
                worst = max(worst, np.abs(out[g, b, h * hd:(h + 1) * hd] - ref[0]).max())
    assert worst < 2e-2, worst


@pytest.mark.parametrize("hd", [64, 128, 72, 96, 104])
@pytest.mark.parametrize("n_keys,splits", [(1, 1), (2, 0), (131, 3), (700, 0), (2049, 32), (300, 1)])
def test_decode_attention_matches_oracle(hd, n_keys, splits):
    G, B, H, P = 2, 3, 2, 2112
    d = H * hd
    q = ki.normal_bf16(8, 0, (G, B, d), 1.0, DEV)
    kc = ki.normal_bf16(8, 1, (G, B, H, P, hd), 1.0, DEV)
    vc = ki.normal_bf16(8, 2, (G, B, H, P, hd), 1.0, DEV)
    kc[:, :, :, n_keys:] = float("nan")   # rows past the sequence must never be read into the result
    vc[:, :, :, n_keys:] = float("nan")
    out = kr.op_decode_attention(q, kc, vc, n_keys, splits).float().cpu().numpy()
    assert not np.isnan(out).any()
    qn, kn, vn = q.float().cpu().numpy(), kc.float().cpu().numpy(), vc.float().cpu().numpy()
    worst = 0.0
    for g in range(G):
        for b in range(B):
            for h in range(H):
                ref = oracle.attention_head(qn[g, b:b + 1, h * hd:(h + 1) * hd], kn[g, b, h, :n_keys],
                                            vn[g, b, h, :n_keys], q_pos0=n_keys - 1)
                worst = max(worst, np.abs(out[g, b, h * hd:(h + 1) * hd] - ref[0]).max())
    assert worst < 2e-2, worst


def test_decode_attention_scratch_checks():
    sp, nb = kr.decode_attention_sizes(4, 16, 2048, 16, 64)
    assert 1 <= sp <= 32 and nb == (0 if sp == 1 else 4 * 16 * 16 * sp * 66 * 4)
    assert kr.decode_attention_sizes(1, 1, 50, 2, 64, 1) == (1, 0)
    q = torch.zeros(1, 1, 128, dtype=torch.bfloat16, device=DEV)
    kc = torch.zeros(1, 1, 2, 64, 64, dtype=torch.bfloat16, device=DEV)
    small = torch.empty(16, dtype=torch.uint8, device=DEV)
    with pytest.raises(kr.KrakenError) as e:
        kr.op_decode_attention(q, kc, kc, 40, splits=4, partials=small)
    assert e.value.status == kr.ECAPACITY


@pytest.mark.parametrize("M", [1, 16, 17, 32])
def test_skinny_gemm_integer_exact(M):
    """The weight-streaming kernel used for decode and the tail (n_tile = 8), ragged N and K."""
    r = gemm_case(3, M, 203 * 8 + 8, 136, kr.EPI_F32, 8, integer=True, seed=6)
    assert np.array_equal(r["out_f32"], r["ref"])


@pytest.mark.parametrize("epi", [kr.EPI_F32, kr.EPI_BF16, kr.EPI_GELU_BF16, kr.EPI_RESID_F32])
def test_skinny_gemm_epilogues(epi):
    r = gemm_case(4, 16, 1024, 4096, epi, 8, seed=7)
    if r["out_f32"] is not None:
        assert np.abs(r["out_f32"] - r["ref"]).max() < 5e-4
    else:
        ok, worst = bf16_ulp_close(r["out_bf16"], r["ref"], ulps=1.0, atol=2e-4)
        assert ok, worst


def test_skinny_gemm_unaligned_output_rows():
    """fp32 output with an odd row stride (the logits of a 50257-word vocabulary)."""
    G, M, Nout, K = 1, 5, 1001, 256
    a = ki.normal_bf16(9, 0, (G, M, K), 1.0, DEV)
    w = ki.normal_bf16(9, 1, (G, Nout, K), 0.06, DEV)
    out = torch.full((M, Nout), float("nan"), dtype=torch.float32, device=DEV)
    args = kr.GemmArgs()
    args.a, args.lda, args.w, args.ldw = a.data_ptr(), K, w.data_ptr(), K
    args.groups, args.m, args.n_out, args.k, args.epilogue, args.n_tile = G, M, Nout, K, kr.EPI_F32, 8
    args.out_f32, args.ld_out_f32 = out.data_ptr(), Nout
    kr.op_grouped_gemm(args)
    ref = oracle.linear(a[0].float().cpu().numpy(), bits(w[0]))
    assert np.abs(out.cpu().numpy() - ref).max() < 2e-4


# ------------------------------------------------------------------ IEEE half image, single steps

def test_half_image_gemm_layernorm_and_attention():
    """The single steps of libkraken_f16.so on half tensors against the oracle's steps in half mode."""
    with kr.storage_dtype("f16"):
        G, M, K, Nout = 2, 300, 256, 384
        a = ki.normal_f16(31, 0, (G, M, K), 1.0, DEV)
        w = ki.normal_f16(31, 1, (G, Nout, K), 0.05, DEV)
        bias = ki.normal_f16(31, 2, (G, Nout), 0.1, DEV)
        out = torch.empty(G, M, Nout, dtype=torch.float32, device=DEV)
        args = kr.GemmArgs()
        args.a, args.a_gstride, args.lda = a.data_ptr(), M * K, K
        args.w, args.w_gstride, args.ldw = w.data_ptr(), Nout * K, K
        args.bias, args.bias_gstride = bias.data_ptr(), Nout
        args.groups, args.m, args.n_out, args.k = G, M, Nout, K
        args.epilogue = kr.EPI_F32
        args.out_f32, args.out_f32_gstride, args.ld_out_f32 = out.data_ptr(), M * Nout, Nout
        kr.op_grouped_gemm(args)
        torch.cuda.synchronize()
        for g in range(G):
            ref = oracle.linear(a[g].float().cpu().numpy(), bits(w[g]), bits(bias[g]), half=True)
            assert np.abs(out[g].cpu().numpy() - ref).max() < 2e-4 * max(1.0, np.abs(ref).max())
        # LayerNorm with half gamma / beta and half output
        x = (ki.normal_bf16(32, 0, (G, 40, 256), 1.0, DEV).float() * 1.5 + 0.2).contiguous()
        gamma = (1 + ki.normal_bf16(32, 1, (G, 256), 0.3, DEV).float()).to(torch.float16)
        beta = ki.normal_f16(32, 2, (G, 256), 0.3, DEV)
        ln = kr.op_layernorm(x, None, gamma, beta)
        assert ln.dtype == torch.float16
        for g in range(G):
            ref = oracle.layernorm(x[g].cpu().numpy(), None, bits(gamma[g]), bits(beta[g]), round_out=True, half=True)
            got = ln[g].float().cpu().numpy()
            assert (np.abs(got - ref) <= 2.0 ** -10 * np.maximum(np.abs(ref), 0.05)).all()
        # attention on half q, k, v
        B, H, hd, P, seqlen = 2, 2, 64, 256, 200
        q = ki.normal_f16(33, 0, (G, B * seqlen, H * hd), 1.0, DEV)
        kc = ki.normal_f16(33, 1, (G, B, H, P, hd), 1.0, DEV)
        vc = ki.normal_f16(33, 2, (G, B, H, P, hd), 1.0, DEV)
        o = kr.op_attention(q, kc, vc, B, seqlen, 0, H).float().cpu().numpy()
        qn, kn, vn = q.float().cpu().numpy(), kc.float().cpu().numpy(), vc.float().cpu().numpy()
        for g in range(G):
            for b in range(B):
                for h in range(H):
                    ref = oracle.attention_head(qn[g, b * seqlen:(b + 1) * seqlen, h * hd:(h + 1) * hd],
                                                kn[g, b, h, :seqlen], vn[g, b, h, :seqlen])
                    assert np.abs(o[g, b * seqlen:(b + 1) * seqlen, h * hd:(h + 1) * hd] - ref).max() < 1e-2
        od = kr.op_decode_attention(q[:, :B].contiguous(), kc, vc, 150).float().cpu().numpy()
        for g in range(G):
            for b in range(B):
                for h in range(H):
                    ref = oracle.attention_head(qn[g, b:b + 1, h * hd:(h + 1) * hd], kn[g, b, h, :150], vn[g, b, h, :150],
                                                q_pos0=149)
                    assert np.abs(od[g, b, h * hd:(h + 1) * hd] - ref[0]).max() < 1e-2

