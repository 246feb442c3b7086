"""Python binding of libkraken.so: argument marshalling only.

Every step of the Kraken prefill / decode path runs inside the CUDA library; this module
turns torch tensors (used purely as device-memory owners) into the pointers and sizes of the
C ABI declared in include/kraken.h.  There is no fallback: without the built library every
call raises.
"""
from __future__ import annotations

import contextlib
import ctypes as C
import os
from typing import Dict, Optional

import torch

from . import build as kbuild

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkraken.so")

OK, EINVAL, EUNSUPPORTED, ECAPACITY, ESTATE, ECUDA = 0, -1, -2, -3, -4, -5
EPI_F32, EPI_BF16, EPI_GELU_BF16, EPI_RESID_F32, EPI_RESID_SUM, EPI_QKV = range(6)

WEIGHT_FIELDS = (
    "wte", "wpe", "ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_proj", "b_proj",
    "ln2_g", "ln2_b", "w_up", "b_up", "w_down", "b_down",
    "w_concat", "b_concat", "lnf_g", "lnf_b",
)

PROF_CATEGORIES = ("embed", "layernorm", "gemm_qkv", "attention", "gemm_proj", "gemm_up", "gemm_down", "tail")
PROF_COUNT = len(PROF_CATEGORIES)

EXPORTS = (
    "kraken_query_sizes", "kraken_create", "kraken_prefill", "kraken_prefill_host",
    "kraken_prefill_all_logits", "kraken_prefill_packed", "kraken_seq_lens", "kraken_logits_rows",
    "kraken_stage_begin", "kraken_stage_begin_decode", "kraken_stage_attention", "kraken_stage_ffn", "kraken_stage_buffers", "kraken_stage_concat",
    "kraken_stage_head", "kraken_decode_step", "kraken_decode_step_host", "kraken_kv_view",
    "kraken_device_status", "kraken_cur_len", "kraken_profile_enable", "kraken_profile_read", "kraken_reset", "kraken_destroy", "kraken_strerror", "kraken_last_cuda_error",
    "kraken_op_embed", "kraken_op_layernorm", "kraken_op_grouped_gemm", "kraken_op_attention",
    "kraken_op_grouped_gemm_ln", "kraken_gemm_ln_scratch_bytes",
    "kraken_op_decode_attention", "kraken_decode_attention_sizes",
    "kraken_op_decode_attention_static", "kraken_decode_attention_static_capacity", "kraken_storage_dtype",
    "kraken_tuning_set", "kraken_test_wait_limit", "kraken_test_mma_issue_rate",
)

TUNE_LN_ROW_KERNEL, TUNE_ATTN_SCHEDULE, TUNE_LN_FUSION, TUNE_LAST_LAYER = 0, 1, 2, 3
STATUS_BAD_TOKEN, STATUS_WAIT_LIMIT = 1, 2


class KrakenConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("n_branch", "n_layer", "d_model", "n_head", "d_ff", "vocab", "max_pos", "max_batch")] + [
        ("ln_eps", C.c_float), ("gelu_tanh", C.c_int32), ("final_ln", C.c_int32), ("n_kv_head", C.c_int32),
        ("no_combine", C.c_int32), ("parallel_ffn", C.c_int32), ("reserved", C.c_int32 * 2)]


class KrakenWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in WEIGHT_FIELDS]


class GemmArgs(C.Structure):
    _fields_ = [
        ("a", C.c_void_p), ("a_gstride", C.c_int64), ("lda", C.c_int32),
        ("w", C.c_void_p), ("w_gstride", C.c_int64), ("ldw", C.c_int32),
        ("bias", C.c_void_p), ("bias_gstride", C.c_int64),
        ("groups", C.c_int32), ("m", C.c_int32), ("n_out", C.c_int32), ("k", C.c_int32),
        ("epilogue", C.c_int32),
        ("out_f32", C.c_void_p), ("out_f32_gstride", C.c_int64), ("ld_out_f32", C.c_int32),
        ("out_bf16", C.c_void_p), ("out_bf16_gstride", C.c_int64), ("ld_out_bf16", C.c_int32),
        ("resid", C.c_void_p), ("resid_gstride", C.c_int64), ("ld_resid", C.c_int32),
        ("sum", C.c_void_p), ("ld_sum", C.c_int32),
        ("k_cache", C.c_void_p), ("v_cache", C.c_void_p), ("cache_gstride", C.c_int64),
        ("seqlen", C.c_int32), ("pos0", C.c_int32), ("n_head", C.c_int32), ("head_dim", C.c_int32),
        ("max_pos", C.c_int32), ("gelu_tanh", C.c_int32), ("n_tile", C.c_int32), ("n_kv_head", C.c_int32),
        ("w_constant", C.c_int32),
    ]


class GemmLnArgs(C.Structure):
    _fields_ = [
        ("ln_out", C.c_void_p), ("ln_out_gstride", C.c_int64), ("ld_ln_out", C.c_int32),
        ("gamma", C.c_void_p), ("beta", C.c_void_p), ("gb_gstride", C.c_int64),
        ("y", C.c_void_p), ("ld_y", C.c_int32),
        ("eps", C.c_float),
        ("d_scratch", C.c_void_p), ("scratch_bytes", C.c_size_t),
    ]


class KrakenError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        detail = lib().kraken_last_cuda_error().decode() if status == ECUDA else ""
        super().__init__(f"{what}: {strerror(status)} ({status})" + (f" [{detail}]" if detail else ""))


_libs: Dict[str, C.CDLL] = {}
_current_dtype = "bf16"
TORCH_DTYPE = {"bf16": torch.bfloat16, "f16": torch.float16}


@contextlib.contextmanager
def storage_dtype(dtype: str):
    """Within the block, calls that do not name a dtype go to that image ('bf16': libkraken.so, 'f16':
    libkraken_f16.so, the same ABI with IEEE half as the 16-bit storage type)."""
    global _current_dtype
    if dtype not in TORCH_DTYPE:
        raise ValueError("storage dtype must be 'bf16' or 'f16'")
    old, _current_dtype = _current_dtype, dtype
    try:
        yield
    finally:
        _current_dtype = old


def lib(dtype: Optional[str] = None) -> C.CDLL:
    """Loads the library image of the storage dtype; raises if it has not been built."""
    dtype = dtype or _current_dtype
    if dtype not in _libs:
        path = kbuild.lib_path(dtype)
        if not os.path.exists(path):
            raise RuntimeError(
                f"{path} is missing: build it with `python -m paper_2408_07802_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        L = C.CDLL(path)
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        L.kraken_query_sizes.argtypes = [C.POINTER(KrakenConfig), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
        L.kraken_create.argtypes = [C.POINTER(KrakenConfig), C.POINTER(KrakenWeights), vp, C.c_size_t, vp,
                                    C.c_size_t, C.POINTER(vp)]
        L.kraken_prefill.argtypes = [vp, vp, i32, i32, vp, vp]
        L.kraken_prefill_host.argtypes = [vp, vp, i32, i32, vp, vp]
        L.kraken_prefill_all_logits.argtypes = [vp, vp, i32, i32, vp, vp]
        L.kraken_prefill_packed.argtypes = [vp, vp, vp, i32, vp, vp]
        L.kraken_seq_lens.argtypes = [vp, vp, i32]
        L.kraken_stage_begin.argtypes = [vp, vp, i32, i32, vp]
        L.kraken_stage_begin_decode.argtypes = [vp, vp, i32, vp]
        L.kraken_stage_attention.argtypes = [vp, i32, vp]
        L.kraken_stage_ffn.argtypes = [vp, i32, vp, vp]
        L.kraken_stage_buffers.argtypes = [vp, C.POINTER(vp), C.POINTER(vp)]
        L.kraken_stage_concat.argtypes = [vp, vp, vp]
        L.kraken_stage_head.argtypes = [vp, vp, vp, vp]
        L.kraken_logits_rows.argtypes = [vp, vp, i32, vp, vp]
        L.kraken_decode_step.argtypes = [vp, vp, i32, vp, vp]
        L.kraken_decode_step_host.argtypes = [vp, vp, i32, vp, vp]
        L.kraken_kv_view.argtypes = [vp, i32, i32, i32, C.POINTER(vp), C.POINTER(i64 * 4)]
        L.kraken_device_status.argtypes = [vp, C.POINTER(C.c_uint32)]
        L.kraken_cur_len.argtypes = [vp, C.POINTER(i32)]
        L.kraken_profile_enable.argtypes = [vp, i32]
        L.kraken_profile_read.argtypes = [vp, C.POINTER(C.c_double * PROF_COUNT), C.POINTER(i64 * PROF_COUNT)]
        L.kraken_reset.argtypes = [vp]
        L.kraken_destroy.argtypes = [vp]
        L.kraken_destroy.restype = None
        L.kraken_strerror.argtypes = [C.c_int]
        L.kraken_strerror.restype = C.c_char_p
        L.kraken_last_cuda_error.argtypes = []
        L.kraken_last_cuda_error.restype = C.c_char_p
        L.kraken_op_embed.argtypes = [vp, i32, i32, i32, vp, vp, i32, i32, vp, vp, vp]
        L.kraken_op_layernorm.argtypes = [vp, i64, vp, vp, vp, i32, i32, i32, C.c_float, vp, vp, vp]
        L.kraken_op_grouped_gemm.argtypes = [C.POINTER(GemmArgs), vp, vp]
        L.kraken_op_grouped_gemm_ln.argtypes = [C.POINTER(GemmArgs), C.POINTER(GemmLnArgs), vp, vp]
        L.kraken_gemm_ln_scratch_bytes.argtypes = [i32, i32, i32, i32, i32, C.POINTER(C.c_size_t)]
        L.kraken_op_attention.argtypes = [vp, i64, vp, vp, i64, i64, i32, i32, i32, i32, i32, i32, i32, i32, vp, i64, vp]
        L.kraken_op_decode_attention.argtypes = [vp, i64, vp, vp, i64, i64, i32, i32, i32, i32, i32, i32, i32, i32, vp,
                                                 C.c_size_t, vp, i64, vp]
        L.kraken_decode_attention_sizes.argtypes = [i32, i32, i32, i32, i32, C.POINTER(i32), C.POINTER(C.c_size_t)]
        L.kraken_op_decode_attention_static.argtypes = [vp, i64, vp, vp, i64, i64, i32, i32, i32, i32, i32, i32, i32,
                                                        vp, i64, vp]
        L.kraken_decode_attention_static_capacity.argtypes = []
        L.kraken_decode_attention_static_capacity.restype = C.c_size_t
        L.kraken_storage_dtype.argtypes = []
        L.kraken_tuning_set.argtypes = [i32, i32]
        L.kraken_test_wait_limit.argtypes = [vp, C.c_uint32, vp]
        L.kraken_test_mma_issue_rate.argtypes = [i32, i32, i32, vp, i32, C.POINTER(C.c_int32), vp, vp]
        if L.kraken_storage_dtype() != (1 if dtype == "f16" else 0):
            raise RuntimeError(f"{path} was not built for storage dtype {dtype}")
        _libs[dtype] = L
    return _libs[dtype]


def strerror(status: int) -> str:
    return lib().kraken_strerror(int(status)).decode()


def _check(status: int, what: str):
    if status != OK:
        raise KrakenError(status, what)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def make_config(shape, max_batch: Optional[int] = None, max_pos: Optional[int] = None, **over) -> KrakenConfig:
    """kraken_config from any object with the hyper-parameter attributes (e.g. kraken_inputs.KrakenShape)."""
    cfg = KrakenConfig(
        n_branch=shape.n_branch, n_layer=shape.n_layer, d_model=shape.d_model, n_head=shape.n_head,
        d_ff=shape.d_ff, vocab=shape.vocab, max_pos=max_pos or shape.max_pos,
        max_batch=max_batch or shape.batch, ln_eps=shape.ln_eps, gelu_tanh=shape.gelu_tanh,
        final_ln=shape.final_ln, n_kv_head=int(getattr(shape, "n_kv_head", 0) or 0),
        no_combine=int(getattr(shape, "no_combine", 0) or 0),
        parallel_ffn=int(getattr(shape, "parallel_ffn", 0) or 0))
    for k, v in over.items():
        setattr(cfg, k, v)
    return cfg


def query_sizes(cfg: KrakenConfig):
    kv, sc = C.c_size_t(0), C.c_size_t(0)
    _check(lib().kraken_query_sizes(C.byref(cfg), C.byref(kv), C.byref(sc)), "kraken_query_sizes")
    return kv.value, sc.value


class KrakenModel:
    """Owns the device buffers (through torch) and a kraken_handle."""

    def __init__(self, cfg: KrakenConfig, weights: Dict[str, Optional[torch.Tensor]], device="cuda:0",
                 dtype: Optional[str] = None):
        self.cfg = cfg
        self.device = torch.device(device)
        self.dtype = dtype or _current_dtype
        for k in WEIGHT_FIELDS:
            t = weights.get(k)
            if t is not None:
                assert t.dtype == TORCH_DTYPE[self.dtype] and t.is_contiguous() and t.device == self.device, k
        self.weights = dict(weights)
        kv_bytes, scratch_bytes = query_sizes(cfg)
        self.kv = torch.empty(kv_bytes, dtype=torch.uint8, device=self.device)
        self.scratch = torch.empty(scratch_bytes, dtype=torch.uint8, device=self.device)
        w = KrakenWeights(**{k: _ptr(weights.get(k)) for k in WEIGHT_FIELDS})
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(lib(self.dtype).kraken_create(C.byref(cfg), C.byref(w), self.kv.data_ptr(), kv_bytes,
                                       self.scratch.data_ptr(), scratch_bytes, C.byref(h)), "kraken_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            lib(self.dtype).kraken_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    # -------- the three calls of the path
    def prefill(self, tokens: torch.Tensor, logits: Optional[torch.Tensor] = None) -> torch.Tensor:
        """tokens: device int32 [batch, seqlen] -> fp32 [batch, V] logits of the last position."""
        b, l = tokens.shape
        assert tokens.dtype == torch.int32 and tokens.is_contiguous() and tokens.device == self.device
        if logits is None:
            logits = torch.empty(b, self.cfg.vocab, dtype=torch.float32, device=self.device)
        _check(lib(self.dtype).kraken_prefill(self._h, tokens.data_ptr(), b, l, logits.data_ptr(), _stream()), "kraken_prefill")
        return logits

    def prefill_host(self, tokens: torch.Tensor, logits: torch.Tensor) -> torch.Tensor:
        """tokens / logits: HOST tensors (pinned for full-rate copies); blocks until the logits are there."""
        b, l = tokens.shape
        assert tokens.dtype == torch.int32 and tokens.device.type == "cpu" and logits.device.type == "cpu"
        _check(lib(self.dtype).kraken_prefill_host(self._h, tokens.data_ptr(), b, l, logits.data_ptr(), _stream()),
               "kraken_prefill_host")
        return logits

    def prefill_all_logits(self, tokens: torch.Tensor) -> torch.Tensor:
        b, l = tokens.shape
        assert tokens.dtype == torch.int32 and tokens.is_contiguous() and tokens.device == self.device
        logits = torch.empty(b, l, self.cfg.vocab, dtype=torch.float32, device=self.device)
        _check(lib(self.dtype).kraken_prefill_all_logits(self._h, tokens.data_ptr(), b, l, logits.data_ptr(), _stream()),
               "kraken_prefill_all_logits")
        return logits

    def prefill_packed(self, tokens: torch.Tensor, seq_lens, logits: Optional[torch.Tensor] = None) -> torch.Tensor:
        """tokens: device int32 [sum(seq_lens)], the sequences back to back -> fp32 [batch, V] logits of every
        sequence's last position."""
        lens = torch.as_tensor(seq_lens, dtype=torch.int32).contiguous()
        b = lens.numel()
        assert tokens.dtype == torch.int32 and tokens.is_contiguous() and tokens.device == self.device
        assert tokens.numel() == int(lens.sum())
        if logits is None:
            logits = torch.empty(b, self.cfg.vocab, dtype=torch.float32, device=self.device)
        _check(lib(self.dtype).kraken_prefill_packed(self._h, tokens.data_ptr(), lens.data_ptr(), b, logits.data_ptr(),
                                                     _stream()), "kraken_prefill_packed")
        return logits

    # -------- the path in pieces, for the branch-parallel deployment (see branch_parallel.py)
    def stage_begin(self, tokens: torch.Tensor):
        b, l = tokens.shape
        assert tokens.dtype == torch.int32 and tokens.is_contiguous() and tokens.device == self.device
        _check(lib(self.dtype).kraken_stage_begin(self._h, tokens.data_ptr(), b, l, _stream()), "kraken_stage_begin")
        self._stage_shape = (b, l)

    def stage_begin_decode(self, tokens: torch.Tensor):
        assert tokens.dtype == torch.int32 and tokens.is_contiguous() and tokens.device == self.device
        _check(lib(self.dtype).kraken_stage_begin_decode(self._h, tokens.data_ptr(), tokens.numel(), _stream()),
               "kraken_stage_begin_decode")
        self._stage_shape = (tokens.numel(), 1)

    def stage_attention(self, layer: int):
        _check(lib(self.dtype).kraken_stage_attention(self._h, layer, _stream()), "kraken_stage_attention")

    def stage_ffn(self, layer: int, y: torch.Tensor):
        assert y.dtype == torch.float32 and y.is_contiguous() and y.device == self.device
        _check(lib(self.dtype).kraken_stage_ffn(self._h, layer, y.data_ptr(), _stream()), "kraken_stage_ffn")

    def stage_buffers(self):
        """(x0, local_sum): fp32 [batch*seqlen, d] views of the shared embedding and of the sum of this
        handle's layer outputs (rewritten by every stage_ffn)."""
        p0, p1 = C.c_void_p(), C.c_void_p()
        _check(lib(self.dtype).kraken_stage_buffers(self._h, C.byref(p0), C.byref(p1)), "kraken_stage_buffers")
        b, l = self._stage_shape
        flat = self.scratch.view(torch.float32)
        base = self.scratch.data_ptr()
        n = b * l * self.cfg.d_model
        return (flat[(p0.value - base) // 4:(p0.value - base) // 4 + n].view(b * l, self.cfg.d_model),
                flat[(p1.value - base) // 4:(p1.value - base) // 4 + n].view(b * l, self.cfg.d_model))

    def stage_concat(self) -> torch.Tensor:
        b, _ = self._stage_shape
        z = torch.empty(b, self.cfg.d_model, dtype=torch.float32, device=self.device)
        _check(lib(self.dtype).kraken_stage_concat(self._h, z.data_ptr(), _stream()), "kraken_stage_concat")
        return z

    def stage_head(self, z: torch.Tensor, logits: Optional[torch.Tensor] = None) -> torch.Tensor:
        b, _ = self._stage_shape
        assert z.dtype == torch.float32 and z.is_contiguous() and z.device == self.device
        if logits is None:
            logits = torch.empty(b, self.cfg.vocab, dtype=torch.float32, device=self.device)
        _check(lib(self.dtype).kraken_stage_head(self._h, z.data_ptr(), logits.data_ptr(), _stream()), "kraken_stage_head")
        return logits

    def seq_lens(self, batch: int):
        out = torch.zeros(batch, dtype=torch.int32)
        _check(lib(self.dtype).kraken_seq_lens(self._h, out.data_ptr(), batch), "kraken_seq_lens")
        return out.tolist()

    def logits_rows(self, rows) -> torch.Tensor:
        rows_t = torch.as_tensor(rows, dtype=torch.int32).contiguous()
        out = torch.empty(rows_t.numel(), self.cfg.vocab, dtype=torch.float32, device=self.device)
        _check(lib(self.dtype).kraken_logits_rows(self._h, rows_t.data_ptr(), rows_t.numel(), out.data_ptr(), _stream()),
               "kraken_logits_rows")
        torch.cuda.current_stream().synchronize()  # rows_t (host) must outlive the copy
        return out

    def decode_step(self, tokens: torch.Tensor, logits: Optional[torch.Tensor] = None) -> torch.Tensor:
        assert tokens.dtype == torch.int32 and tokens.is_contiguous() and tokens.device == self.device
        b = tokens.numel()
        if logits is None:
            logits = torch.empty(b, self.cfg.vocab, dtype=torch.float32, device=self.device)
        _check(lib(self.dtype).kraken_decode_step(self._h, tokens.data_ptr(), b, logits.data_ptr(), _stream()),
               "kraken_decode_step")
        return logits

    def decode_step_host(self, tokens: torch.Tensor, logits: torch.Tensor) -> torch.Tensor:
        """tokens [batch] / logits [batch, V]: HOST tensors; blocks until the logits are there."""
        assert tokens.dtype == torch.int32 and tokens.device.type == "cpu" and logits.device.type == "cpu"
        _check(lib(self.dtype).kraken_decode_step_host(self._h, tokens.data_ptr(), tokens.numel(), logits.data_ptr(),
                                             _stream()), "kraken_decode_step_host")
        return logits

    # -------- inspection
    def kv_view(self, layer: int, branch: int, which: int) -> torch.Tensor:
        """bf16 view [max_batch, key/value heads, max_pos, head_dim] of the K (0) or V (1) cache of (layer, branch)."""
        p = C.c_void_p()
        st = (C.c_int64 * 4)()
        _check(lib(self.dtype).kraken_kv_view(self._h, layer, branch, which, C.byref(p), C.byref(st)), "kraken_kv_view")
        c = self.cfg
        hd = c.d_model // c.n_head
        off = (p.value - self.kv.data_ptr()) // 2
        flat = self.kv.view(TORCH_DTYPE[self.dtype])
        return flat.as_strided((c.max_batch, c.n_kv_head or c.n_head, c.max_pos, hd), tuple(st), off)

    def device_status(self) -> int:
        f = C.c_uint32(0)
        _check(lib(self.dtype).kraken_device_status(self._h, C.byref(f)), "kraken_device_status")
        return f.value

    @property
    def cur_len(self) -> int:
        v = C.c_int32(0)
        _check(lib(self.dtype).kraken_cur_len(self._h, C.byref(v)), "kraken_cur_len")
        return v.value

    def profile_enable(self, on: bool):
        _check(lib(self.dtype).kraken_profile_enable(self._h, int(on)), "kraken_profile_enable")

    def profile_read(self):
        """({category: device ms}, {category: launches}) since the last read; synchronises."""
        ms = (C.c_double * PROF_COUNT)()
        n = (C.c_int64 * PROF_COUNT)()
        _check(lib(self.dtype).kraken_profile_read(self._h, C.byref(ms), C.byref(n)), "kraken_profile_read")
        return dict(zip(PROF_CATEGORIES, list(ms))), dict(zip(PROF_CATEGORIES, list(n)))

    def reset(self):
        _check(lib(self.dtype).kraken_reset(self._h), "kraken_reset")


# ------------------------------------------------------------------ single steps

def op_embed(ids: torch.Tensor, seqlen: int, pos0: int, wte: torch.Tensor, wpe: torch.Tensor,
             status: Optional[torch.Tensor] = None) -> torch.Tensor:
    n = ids.numel()
    d = wte.shape[1]
    out = torch.empty(n, d, dtype=torch.float32, device=ids.device)
    _check(lib().kraken_op_embed(ids.data_ptr(), n, seqlen, pos0, wte.data_ptr(), wpe.data_ptr(), d, wte.shape[0],
                                 out.data_ptr(), _ptr(status), _stream()), "kraken_op_embed")
    return out


def op_layernorm(a: torch.Tensor, y: Optional[torch.Tensor], gamma: torch.Tensor, beta: Optional[torch.Tensor],
                 eps: float = 1e-5, shared_a: bool = False, status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """a fp32 [G, rows, d] (or [rows, d] with shared_a, used by every group); gamma [G, d]; status: device
    uint32 word (with it, many-row calls take the persistent kernel)."""
    G, d = gamma.shape
    rows = a.shape[-2]
    out = torch.empty(G, rows, d, dtype=gamma.dtype, device=a.device)
    _check(lib().kraken_op_layernorm(a.data_ptr(), 0 if shared_a else rows * d, _ptr(y), gamma.data_ptr(),
                                     _ptr(beta), G, rows, d, eps, out.data_ptr(), _ptr(status), _stream()),
           "kraken_op_layernorm")
    return out


def op_grouped_gemm(args: GemmArgs, status: Optional[torch.Tensor] = None):
    _check(lib().kraken_op_grouped_gemm(C.byref(args), _ptr(status), _stream()), "kraken_op_grouped_gemm")


def gemm_ln_scratch_bytes(groups: int, m: int, n_out: int, k: int, n_tile: int = 0) -> int:
    n = C.c_size_t(0)
    _check(lib().kraken_gemm_ln_scratch_bytes(groups, m, n_out, k, n_tile, C.byref(n)), "kraken_gemm_ln_scratch_bytes")
    return int(n.value)


def op_grouped_gemm_ln(args: GemmArgs, ln: GemmLnArgs, status: Optional[torch.Tensor] = None):
    """A RESID_F32 / RESID_SUM grouped GEMM with the LayerNorm of the finished rows in the same kernel."""
    _check(lib().kraken_op_grouped_gemm_ln(C.byref(args), C.byref(ln), _ptr(status), _stream()),
           "kraken_op_grouped_gemm_ln")


def op_attention(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, batch: int, seqlen: int, pos0: int,
                 n_head: int) -> torch.Tensor:
    """q bf16 [G, batch*seqlen, d]; k_cache / v_cache bf16 [G, batch, key/value heads, max_pos, head_dim]
    (fewer key/value heads than n_head = grouped-query attention)."""
    G, _, d = q.shape
    _, _, Hkv, P, hd = k_cache.shape
    assert n_head % Hkv == 0 and n_head * hd == d
    out = torch.empty_like(q)
    _check(lib().kraken_op_attention(q.data_ptr(), q.stride(0), k_cache.data_ptr(), v_cache.data_ptr(),
                                     k_cache.stride(0), k_cache.stride(1), G, batch, seqlen, pos0, n_head, Hkv, hd, P,
                                     out.data_ptr(), out.stride(0), _stream()), "kraken_op_attention")
    return out


def decode_attention_sizes(groups: int, batch: int, n_keys: int, n_head: int, head_dim: int, splits: int = 0):
    """(splits, scratch bytes) for op_decode_attention."""
    sp, nb = C.c_int32(splits), C.c_size_t(0)
    _check(lib().kraken_decode_attention_sizes(groups, batch, n_keys, n_head, head_dim, C.byref(sp), C.byref(nb)),
           "kraken_decode_attention_sizes")
    return sp.value, nb.value


def op_decode_attention(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, n_keys: int,
                        splits: int = 0, partials: Optional[torch.Tensor] = None) -> torch.Tensor:
    """q bf16 [G, batch, d]; caches bf16 [G, batch, key/value heads, max_pos, head_dim]; attends to rows
    0..n_keys-1.  The number of query heads is d / head_dim."""
    G, B, d = q.shape
    _, _, Hkv, P, hd = k_cache.shape
    H = d // hd
    splits, nbytes = decode_attention_sizes(G, B, n_keys, H, hd, splits)
    if partials is None and nbytes:
        partials = torch.empty(nbytes, dtype=torch.uint8, device=q.device)
    out = torch.empty_like(q)
    _check(lib().kraken_op_decode_attention(q.data_ptr(), q.stride(0), k_cache.data_ptr(), v_cache.data_ptr(),
                                            k_cache.stride(0), k_cache.stride(1), G, B, n_keys, H, Hkv, hd, P, splits,
                                            _ptr(partials), 0 if partials is None else partials.numel(),
                                            out.data_ptr(), out.stride(0), _stream()), "kraken_op_decode_attention")
    return out


def op_decode_attention_static(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, n_keys: int,
                               splits: int = 0, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """op_decode_attention for callers that cannot provide scratch: the partials live in a fixed
    array inside the library (see kraken_op_decode_attention_static).  The output tensor is still the
    caller's; this wrapper creates it with torch only when `out` is not given."""
    G, B, d = q.shape
    _, _, H, P, hd = k_cache.shape
    if H * hd != d:
        raise ValueError("kraken_op_decode_attention_static has no grouped-query form: the cache must hold one "
                         f"key/value head per query head (cache heads {H} x head_dim {hd} != d {d})")
    if out is None:
        out = torch.empty_like(q)
    _check(lib().kraken_op_decode_attention_static(q.data_ptr(), q.stride(0), k_cache.data_ptr(), v_cache.data_ptr(),
                                                   k_cache.stride(0), k_cache.stride(1), G, B, n_keys, H, hd, P,
                                                   splits, out.data_ptr(), out.stride(0), _stream()),
           "kraken_op_decode_attention_static")
    return out


def decode_attention_static_capacity() -> int:
    return int(lib().kraken_decode_attention_static_capacity())


def set_tuning(key: int, value: int) -> None:
    """Test / measurement hook: forces one of two equivalent kernels for a step (0 = the library's choice)."""
    _check(lib().kraken_tuning_set(int(key), int(value)), "kraken_tuning_set")


@contextlib.contextmanager
def tuning(key: int, value: int):
    set_tuning(key, value)
    try:
        yield
    finally:
        set_tuning(key, 0)


def test_wait_limit(status: torch.Tensor, limit_us: int) -> None:
    """Launches the probe whose bounded wait runs out after limit_us microseconds and raises bit 1 of `status`
    (a device int32/uint32 word)."""
    _check(lib().kraken_test_wait_limit(status.data_ptr(), int(limit_us), _stream()), "kraken_test_wait_limit")


test_wait_limit.__test__ = False   # not a pytest case


def mma_issue_rate(form: int, issuers: int = 1, iters: int = 2000, n_ctas: int = 148) -> float:
    """SM clock cycles per tcgen05.mma (M 128, K 16) of the issue-rate probe, averaged over the CTAs
    (see kraken_test_mma_issue_rate for the forms)."""
    dev = torch.device("cuda", torch.cuda.current_device())
    cycles = torch.zeros(n_ctas, dtype=torch.int64, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    per = C.c_int32(0)
    _check(lib().kraken_test_mma_issue_rate(form, issuers, iters, cycles.data_ptr(), n_ctas, C.byref(per),
                                            status.data_ptr(), _stream()), "kraken_test_mma_issue_rate")
    torch.cuda.synchronize()
    if int(status.item()) != 0 or bool((cycles < 0).any()):
        raise KrakenError(ECUDA, "kraken_test_mma_issue_rate: a bounded wait gave up")
    return float(cycles.double().mean().item()) / (iters * per.value * issuers)
