"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, and its argument validation / size arithmetic behave as documented."""
import ctypes as C
import os
import re

import pytest

import kraken_inputs as ki
import paper_2408_07802_b200 as kr
from paper_2408_07802_b200 import build as kbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    kbuild.build()
    return kr.lib()


def test_exports_match_header(L):
    text = open(os.path.join(ROOT, "include", "kraken.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(kraken_[a-z_0-9]+)\s*\(", text))
    assert declared == set(kr.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name
    # the IEEE-half image has the same ABI and says which one it is
    kbuild.build(dtype="f16")
    L16 = kr.lib("f16")
    for name in declared:
        assert hasattr(L16, name), name
    assert L.kraken_storage_dtype() == 0 and L16.kraken_storage_dtype() == 1


def test_struct_sizes_match_header():
    # 8 int32 + float + 3 int32 + 4 reserved = 16 words; 18 pointers
    assert C.sizeof(kr.KrakenConfig) == 64
    assert C.sizeof(kr.KrakenWeights) == 18 * 8


def test_query_sizes_arithmetic(L):
    for name, s in ki.CONFIGS.items():
        cfg = kr.make_config(s)
        kv, scratch = kr.query_sizes(cfg)
        assert kv == s.n_layer * s.n_branch * 2 * s.batch * s.max_pos * s.kv_heads * s.head_dim * 2
        T = s.batch * s.max_pos
        floor = T * s.d_model * 4 * (2 + 2 * s.n_branch) + T * s.n_branch * 2 * (3 * s.d_model + s.d_ff)
        # small fixed parts on top: staging, split-KV partials, and the 4 MiB floor of the fused LayerNorm's statistics
        assert floor <= scratch < floor * 1.05 + (1 << 23)
    # grouped-query attention shrinks the cache by the group size (the mitigation of Sec. 4.2)
    full = kr.query_sizes(kr.make_config(ki.CONFIGS["C4"]))[0]
    assert kr.query_sizes(kr.make_config(ki.CONFIGS["C4-gqa4"]))[0] * 4 == full
    assert kr.query_sizes(kr.make_config(ki.CONFIGS["C4-mqa"]))[0] * 16 == full
    # C3's cache is the 8.59 GB the shape implies
    assert abs(kr.query_sizes(kr.make_config(ki.CONFIGS["C3"]))[0] / 1e9 - 8.59) < 0.01


def test_config_validation(L):
    s = ki.CONFIGS["C0"]
    kv, sc = C.c_size_t(), C.c_size_t()
    q = lambda cfg: L.kraken_query_sizes(C.byref(cfg), C.byref(kv), C.byref(sc))
    assert q(kr.make_config(s)) == kr.OK
    assert L.kraken_query_sizes(None, C.byref(kv), C.byref(sc)) == kr.EINVAL
    assert L.kraken_query_sizes(C.byref(kr.make_config(s)), None, None) == kr.EINVAL
    assert q(kr.make_config(s, n_branch=0)) == kr.EINVAL
    assert q(kr.make_config(s, n_head=3)) == kr.EINVAL            # 128 % 3 != 0
    assert q(kr.make_config(s, n_head=4)) == kr.EUNSUPPORTED      # head_dim 32
    assert q(kr.make_config(s, d_ff=100)) == kr.EUNSUPPORTED
    assert q(kr.make_config(s, ln_eps=0.0)) == kr.EINVAL
    assert q(kr.make_config(s, n_kv_head=3)) == kr.EINVAL         # 2 heads cannot share 3 key/value heads
    assert q(kr.make_config(s, n_kv_head=1)) == kr.OK             # multi-query attention


def test_create_rejects_bad_arguments_before_touching_the_device(L):
    cfg = kr.make_config(ki.CONFIGS["C0"])
    w = kr.KrakenWeights()
    h = C.c_void_p()
    assert L.kraken_create(C.byref(cfg), None, 256, 1, 256, 1, C.byref(h)) == kr.EINVAL
    assert L.kraken_create(C.byref(cfg), C.byref(w), 256, 1 << 40, 256, 1 << 40, C.byref(h)) == kr.EINVAL  # null weights
    for f in kr.WEIGHT_FIELDS:
        setattr(w, f, 4096)
    assert L.kraken_create(C.byref(cfg), C.byref(w), 256, 16, 256, 1 << 40, C.byref(h)) == kr.ECAPACITY
    assert L.kraken_create(C.byref(cfg), C.byref(w), 257, 1 << 40, 256, 1 << 40, C.byref(h)) == kr.EINVAL  # alignment
    assert L.kraken_prefill(None, None, 1, 1, None, None) == kr.EINVAL
    assert L.kraken_decode_step(None, None, 1, None, None) == kr.EINVAL
    L.kraken_destroy(None)


def test_strerror(L):
    for code in (0, -1, -2, -3, -4, -5):
        assert len(kr.strerror(code)) > 1
    assert "unknown" in kr.strerror(-99)


def test_gemm_op_validation(L):
    g = kr.GemmArgs()
    assert L.kraken_op_grouped_gemm(None, None, None) == kr.EINVAL
    assert L.kraken_op_grouped_gemm(C.byref(g), None, None) == kr.EINVAL
    g.a, g.w, g.groups, g.m, g.n_out, g.k, g.lda, g.ldw = 4096, 8192, 1, 8, 8, 64, 64, 64
    g.epilogue = kr.EPI_RESID_SUM
    assert L.kraken_op_grouped_gemm(C.byref(g), None, None) == kr.EINVAL   # missing outputs
    g.epilogue = 17
    assert L.kraken_op_grouped_gemm(C.byref(g), None, None) == kr.EINVAL
