"""The scratch-free decode-attention entry point against the one that takes caller scratch.

Runs last in the suite (file name) so that a failure here cannot hide another test's result; it also
passes on its own in a fresh process, where its first call is the one that looks up the address of
the library's built-in partials array.
"""
import ctypes as C

import pytest
import torch

import kraken_inputs as ki
import paper_2408_07802_b200 as kr

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _inputs(G, B, H, hd, P, seed):
    q = ki.normal_bf16(seed, 0, (G, B, H * hd), 1.0, DEV)
    kc = ki.normal_bf16(seed, 1, (G, B, H, P, hd), 1.0, DEV)
    vc = ki.normal_bf16(seed, 2, (G, B, H, P, hd), 1.0, DEV)
    return q, kc, vc


def test_static_scratch_matches_caller_scratch_twice_in_a_row():
    """Two back-to-back calls with different shapes share the built-in array; each must equal the
    existing entry point run on the same inputs (same kernels, same split count: bit for bit, which is
    inside the 2e-2 absolute bound the attention tests use against the oracle)."""
    cases = [(2, 3, 2, 64, 600, 577, 5, 21), (1, 2, 4, 128, 300, 300, 3, 22)]
    for G, B, H, hd, P, n_keys, splits, seed in cases:
        q, kc, vc = _inputs(G, B, H, hd, P, seed)
        out = torch.empty_like(q)           # inputs and output stay the caller's
        rc = kr.lib().kraken_op_decode_attention_static(
            q.data_ptr(), q.stride(0), kc.data_ptr(), vc.data_ptr(), kc.stride(0), kc.stride(1), G, B, n_keys, H,
            hd, P, splits, out.data_ptr(), out.stride(0), torch.cuda.current_stream().cuda_stream)
        assert rc == kr.OK, kr.strerror(rc)
        ref = kr.op_decode_attention(q, kc, vc, n_keys, splits)
        torch.cuda.synchronize()
        assert torch.isfinite(out.float()).all()
        assert (out.float() - ref.float()).abs().max().item() <= 2e-2
        assert torch.equal(out, ref)


def test_static_scratch_rejects_what_does_not_fit():
    cap = kr.decode_attention_static_capacity()
    assert cap == 8 << 20
    G, B, H, hd, P = 4, 64, 16, 128, 64
    q = torch.zeros(G, B, H * hd, dtype=torch.bfloat16, device=DEV)
    kc = torch.zeros(G, B, H, P, hd, dtype=torch.bfloat16, device=DEV)
    need = G * B * H * 8 * (hd + 2) * 4
    assert need > cap
    with pytest.raises(kr.KrakenError) as e:
        kr.op_decode_attention_static(q, kc, kc, 64, splits=8)
    assert e.value.status == kr.ECAPACITY
    # one split needs no partials at all and is always accepted
    out = kr.op_decode_attention_static(q, kc, kc, 64, splits=1)
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()
