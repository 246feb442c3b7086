"""ctypes binding of the plain CPU oracle (test infrastructure, not a product path).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It compiles `kraken_oracle.c` with gcc on first use.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kraken_oracle.c")
_LIB = os.path.join(_HERE, "libkraken_oracle.so")

WEIGHT_FIELDS = (
    "wte", "wpe", "ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_proj", "b_proj",
    "ln2_g", "ln2_b", "w_up", "b_up", "w_down", "b_down",
    "w_concat", "b_concat", "lnf_g", "lnf_b",
)


def build(force: bool = False) -> str:
    """Compile the oracle into a shared library next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fno-fast-math", "-ffp-contract=off",
               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class KoConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("n_branch", "n_layer", "d_model", "n_head", "d_ff", "vocab", "max_pos")] + [
        ("ln_eps", C.c_float), ("gelu_tanh", C.c_int32), ("final_ln", C.c_int32),
        ("bf16_store", C.c_int32), ("y_zero", C.c_int32), ("half", C.c_int32), ("parallel_ffn", C.c_int32),
        ("n_kv_head", C.c_int32)]


class KoWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in WEIGHT_FIELDS]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        L.ko_create.restype = C.c_void_p
        L.ko_create.argtypes = [C.POINTER(KoConfig), C.POINTER(KoWeights)]
        L.ko_destroy.argtypes = [C.c_void_p]
        L.ko_prefill.restype = C.c_int
        L.ko_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_void_p]
        L.ko_decode_step.restype = C.c_int
        L.ko_decode_step.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
        L.ko_cache_ptr.restype = C.POINTER(C.c_float)
        L.ko_cache_ptr.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int]
        L.ko_cur_len.restype = C.c_int
        L.ko_cur_len.argtypes = [C.c_void_p]
        L.ko_gelu.restype = C.c_float
        L.ko_gelu.argtypes = [C.c_float, C.c_int]
        L.ko_round_bf16.restype = C.c_float
        L.ko_round_bf16.argtypes = [C.c_float]
        L.ko_round_f16.restype = C.c_float
        L.ko_round_f16.argtypes = [C.c_float]
        L.ko_f16_to_f32.restype = C.c_float
        L.ko_f16_to_f32.argtypes = [C.c_uint16]
        L.ko_set_half.argtypes = [C.c_int]
        L.ko_num_threads.restype = C.c_int
        L.ko_layernorm.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                   C.c_float, C.c_int, C.c_void_p]
        L.ko_linear.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int64, C.c_void_p,
                                C.c_int, C.c_void_p]
        L.ko_attention_head.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_int64,
                                        C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int64]
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _bits(a) -> Optional[np.ndarray]:
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "weights are passed as bf16 bit patterns (uint16)"
    return a


# ------------------------------------------------------------------ steps

def gelu(x: float, tanh_form: bool = False) -> float:
    return float(lib().ko_gelu(float(x), int(tanh_form)))


def round_bf16(x: float) -> float:
    return float(lib().ko_round_bf16(float(x)))


def round_f16(x: float) -> float:
    """fp32 -> nearest IEEE half (ties to even), as a float."""
    return float(lib().ko_round_f16(float(x)))


def f16_to_f32(bits: int) -> float:
    return float(lib().ko_f16_to_f32(int(bits)))


def num_threads() -> int:
    return int(lib().ko_num_threads())


def layernorm(a, b, gamma_bits, beta_bits, eps=1e-5, round_out=False, half=False) -> np.ndarray:
    """half: the bit patterns (and the rounding of the output) are IEEE half instead of bfloat16."""
    a = _f32(a)
    b = None if b is None else _f32(b)
    rows, d = a.shape
    out = np.empty_like(a)
    g, be = _bits(gamma_bits), _bits(beta_bits)
    lib().ko_set_half(int(half))
    lib().ko_layernorm(_ptr(a), _ptr(b), rows, d, _ptr(g), _ptr(be), eps, int(round_out), _ptr(out))
    lib().ko_set_half(0)
    return out


def linear(x, w_bits, bias_bits=None, half=False) -> np.ndarray:
    x = _f32(x)
    w = _bits(w_bits)
    rows, n_in = x.shape
    n_out = w.shape[0]
    assert w.shape[1] == n_in
    out = np.empty((rows, n_out), dtype=np.float32)
    lib().ko_set_half(int(half))
    lib().ko_linear(_ptr(x), rows, n_in, _ptr(w), n_in, _ptr(_bits(bias_bits)), n_out, _ptr(out))
    lib().ko_set_half(0)
    return out


def attention_head(q, k, v, q_pos0: int = 0) -> np.ndarray:
    """q [n_q, hd] at positions q_pos0.., k/v [>= q_pos0 + n_q, hd]."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    n_q, hd = q.shape
    out = np.empty_like(q)
    lib().ko_attention_head(_ptr(q), hd, _ptr(k), _ptr(v), hd, n_q, q_pos0, hd, _ptr(out), hd)
    return out


# ------------------------------------------------------------------ model

class Oracle:
    """One sequence's Kraken forward state (weights borrowed, KV cache owned)."""

    def __init__(self, shape, weights_bits: Dict[str, Optional[np.ndarray]], bf16_store: bool = False,
                 y_zero: bool = False, final_ln: Optional[bool] = None, gelu_tanh: Optional[bool] = None,
                 half: bool = False):
        self.cfg = KoConfig(
            n_branch=shape.n_branch, n_layer=shape.n_layer, d_model=shape.d_model, n_head=shape.n_head,
            d_ff=shape.d_ff, vocab=shape.vocab, max_pos=shape.max_pos, ln_eps=shape.ln_eps,
            gelu_tanh=int(shape.gelu_tanh if gelu_tanh is None else gelu_tanh),
            final_ln=int(shape.final_ln if final_ln is None else final_ln),
            bf16_store=int(bf16_store), y_zero=int(y_zero or getattr(shape, "no_combine", 0)), half=int(half),
            parallel_ffn=int(getattr(shape, "parallel_ffn", 0)), n_kv_head=int(getattr(shape, "n_kv_head", 0)))
        self._keep = {k: _bits(v) for k, v in weights_bits.items()}
        self.w = KoWeights(**{k: _ptr(self._keep.get(k)) for k in WEIGHT_FIELDS})
        self.shape = shape
        self._h = lib().ko_create(C.byref(self.cfg), C.byref(self.w))
        if not self._h:
            raise ValueError("ko_create rejected the configuration")

    def close(self):
        if self._h:
            lib().ko_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    @property
    def cur_len(self) -> int:
        return lib().ko_cur_len(self._h)

    def prefill(self, ids, logits_from: int = 0, want_layer_out: bool = False):
        """Returns (logits [l - logits_from, V], layer_out [L, N, l, d] or None)."""
        ids = np.ascontiguousarray(ids, dtype=np.int32).reshape(-1)
        l = ids.shape[0]
        s = self.shape
        logits = np.empty((l - logits_from, s.vocab), dtype=np.float32)
        lo = np.empty((s.n_layer, s.n_branch, l, s.d_model), dtype=np.float32) if want_layer_out else None
        rc = lib().ko_prefill(self._h, _ptr(ids), l, _ptr(logits), logits_from, _ptr(lo))
        if rc != 0:
            raise RuntimeError(f"ko_prefill failed: {rc}")
        return logits, lo

    def decode_step(self, token_id: int) -> np.ndarray:
        logits = np.empty((self.shape.vocab,), dtype=np.float32)
        rc = lib().ko_decode_step(self._h, int(token_id), _ptr(logits))
        if rc != 0:
            raise RuntimeError(f"ko_decode_step failed: {rc}")
        return logits

    def cache(self, layer: int, branch: int, which: int) -> np.ndarray:
        """K (which=0) or V (which=1) rows as [key/value heads, cur_len, hd] fp32 (copy)."""
        s = self.shape
        hd = s.head_dim
        n_kv = getattr(s, "n_kv_head", 0) or s.n_head
        out = np.empty((n_kv, self.cur_len, hd), dtype=np.float32)
        for h in range(n_kv):
            p = lib().ko_cache_ptr(self._h, layer, branch, which, h)
            arr = np.ctypeslib.as_array(p, shape=(s.max_pos, hd))
            out[h] = arr[: self.cur_len]
        return out
