"""Seeded synthetic inputs for Kraken prefill/decode workloads.

This module serves both the CPU oracle and the CUDA path.  It holds no model
arithmetic: only workload shapes and a counter-based generator that maps
(seed, tensor id, element index) to a value with integer operations and one
table gather, so the same bits come out on any device torch runs on.

Workloads follow the paper's TTFT experiments (random weights, half precision,
fixed context, uniform token ids; Sec. 4.2) at the five benchmark shapes.
"""
from __future__ import annotations

from dataclasses import dataclass, asdict
from typing import Dict, Optional

import numpy as np
import torch

_M32 = 0xFFFFFFFF

# Field order of the weight set; the position in this tuple is the tensor id
# used to key the generator.
WEIGHT_FIELDS = (
    "wte", "wpe",
    "ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_proj", "b_proj",
    "ln2_g", "ln2_b", "w_up", "b_up", "w_down", "b_down",
    "w_concat", "b_concat", "lnf_g", "lnf_b",
)
TOKENS_TENSOR_ID = 100


@dataclass(frozen=True)
class KrakenShape:
    """Hyper-parameters of one Kraken model plus the request shape.

    n_branch is the paper's degree of parallelism N (Sec. 3.1); n_head is per
    sub-layer (Table 3 caption); d_ff is the FFN hidden width.
    """
    name: str
    n_branch: int
    n_layer: int
    d_model: int
    n_head: int
    d_ff: int
    vocab: int
    max_pos: int
    batch: int
    seqlen: int
    decode_steps: int = 0
    ln_eps: float = 1e-5
    gelu_tanh: int = 0
    final_ln: int = 1
    n_kv_head: int = 0      # key/value heads per sub-layer; 0 = n_head (multi-head), 1 = multi-query
    no_combine: int = 0     # 1: no cross-branch term; with one branch, the standard pre-LN Transformer's layers
    parallel_ffn: int = 0   # 1: out = x + MHA(LN(x)) + FFN(LN(x)): the parallel Attention + FeedForward variant

    @property
    def head_dim(self) -> int:
        return self.d_model // self.n_head

    @property
    def kv_heads(self) -> int:
        return self.n_kv_head or self.n_head

    @property
    def qkv_width(self) -> int:
        """Output width of the fused q | k | v projection: d + 2 * kv_heads * head_dim."""
        return self.d_model + 2 * self.kv_heads * self.head_dim

    def asdict(self):
        return asdict(self)


CONFIGS: Dict[str, KrakenShape] = {
    "C0": KrakenShape("C0", 2, 4, 128, 2, 512, 4096, 128, 1, 128),
    "C1": KrakenShape("C1", 2, 12, 768, 12, 3072, 50257, 1024, 1, 512),
    "C2": KrakenShape("C2", 4, 24, 1024, 16, 4096, 50257, 1024, 1, 1024),
    "C3": KrakenShape("C3", 4, 32, 2048, 16, 8192, 50257, 2048, 4, 2048),
    "C4": KrakenShape("C4", 4, 24, 1024, 16, 4096, 50257, 2176, 16, 2048, decode_steps=128),
    # C4 with grouped-query (4 query heads per key/value head) and multi-query attention: the mitigation
    # the paper names for the KV cache that grows with the number of branches (Sec. 4.2)
    "C4-gqa4": KrakenShape("C4-gqa4", 4, 24, 1024, 16, 4096, 50257, 2176, 16, 2048, decode_steps=128, n_kv_head=4),
    "C4-mqa": KrakenShape("C4-mqa", 4, 24, 1024, 16, 4096, 50257, 2176, 16, 2048, decode_steps=128, n_kv_head=1),
    "C0-gqa": KrakenShape("C0-gqa", 2, 4, 256, 4, 512, 4096, 160, 2, 128, n_kv_head=2),
    "C0-mqa": KrakenShape("C0-mqa", 2, 3, 256, 4, 512, 4096, 160, 1, 150, n_kv_head=1),
}


def _engine(name, n_branch, n_layer, d_model, n_head):
    """Engine shape of the paper's TTFT experiments (Table 3 and Sec. 4.2): FFN width 2 d, vocabulary
    51,200, input context up to 2048, batch 1.  Heads are per sub-layer."""
    return KrakenShape(name, n_branch, n_layer, d_model, n_head, 2 * d_model, 51200, 2048, 1, 2048)


# Table 3, 4-way and 8-way Kraken columns.  The two largest sizes were run by the paper with a quarter
# of their layers (80 -> 20, 96 -> 24), which is what the "q" in the name records.
CONFIGS.update({
    "K1.3B-4": _engine("K1.3B-4", 4, 24, 1248, 12),       # head dim 104
    "K1.3B-8": _engine("K1.3B-8", 8, 24, 960, 10),        # 96
    "K6.7B-4": _engine("K6.7B-4", 4, 32, 2496, 24),       # 104
    "K6.7B-8": _engine("K6.7B-8", 8, 32, 1920, 20),       # 96
    "K13B-4": _engine("K13B-4", 4, 40, 3120, 30),         # 104
    "K13B-8": _engine("K13B-8", 8, 40, 2304, 32),         # 72
    "K65Bq-4": _engine("K65Bq-4", 4, 20, 4992, 39),       # 128
    "K65Bq-8": _engine("K65Bq-8", 8, 20, 3648, 38),       # 96
    "K175Bq-4": _engine("K175Bq-4", 4, 24, 7424, 58),     # 128
    "K175Bq-8": _engine("K175Bq-8", 8, 24, 5472, 57),     # 96
    # small models with the same head dims and FFN ratio, for element-by-element parity runs
    "K0-104": KrakenShape("K0-104", 2, 3, 416, 4, 832, 1024, 320, 2, 300),
    "K0-96": KrakenShape("K0-96", 4, 2, 192, 2, 384, 1024, 320, 1, 200),
    "K0-72": KrakenShape("K0-72", 2, 2, 288, 4, 576, 1024, 320, 1, 257),
    # the standard Transformers of the same table (one branch, no cross-branch term, FFN 4 d): the architecture
    # the paper compares Kraken against, here on the same kernels and the same single GPU
    "S1.3B": KrakenShape("S1.3B", 1, 24, 2048, 16, 8192, 51200, 2048, 1, 2048, no_combine=1),
    "S6.7B": KrakenShape("S6.7B", 1, 32, 4096, 32, 16384, 51200, 2048, 1, 2048, no_combine=1),
    "S0": KrakenShape("S0", 1, 3, 256, 4, 1024, 1024, 160, 2, 100, no_combine=1),
    # and the parallel Attention + FeedForward variants of the same sizes (GPT-J-like dataflow, Sec. 4.2)
    "P1.3B": KrakenShape("P1.3B", 1, 24, 2048, 16, 8192, 51200, 2048, 1, 2048, no_combine=1, parallel_ffn=1),
    "P6.7B": KrakenShape("P6.7B", 1, 32, 4096, 32, 16384, 51200, 2048, 1, 2048, no_combine=1, parallel_ffn=1),
    "P0": KrakenShape("P0", 1, 3, 256, 4, 1024, 1024, 160, 2, 100, no_combine=1, parallel_ffn=1),
})

# TTFT in ms printed by the paper for the Kraken engines (Tables 4 and 5; fp16, batch 1, on as many
# A100-40GB GPUs as the model has branches): {config: {context: ms}}.  Another machine: context only.
PAPER_TTFT_MS = {
    "K1.3B-4": {128: 3.3, 2048: 13.2}, "K6.7B-4": {128: 5.8, 2048: 38.0}, "K13B-4": {128: 10.7, 2048: 66.9},
    "K65Bq-4": {128: 8.5, 2048: 63.8}, "K175Bq-4": {128: 19.9, 2048: 158.9},
    "K1.3B-8": {128: 3.2, 2048: 9.7}, "K6.7B-8": {128: 4.7, 2048: 27.6}, "K13B-8": {128: 6.7, 2048: 42.6},
    "K65Bq-8": {128: 6.2, 2048: 42.9}, "K175Bq-8": {128: 12.4, 2048: 98.0},
}


def weight_shapes(s: KrakenShape) -> Dict[str, tuple]:
    L, N, d, F, V, P = s.n_layer, s.n_branch, s.d_model, s.d_ff, s.vocab, s.max_pos
    return {
        "wte": (V, d), "wpe": (P, d),
        "ln1_g": (L, N, d), "ln1_b": (L, N, d),
        "w_qkv": (L, N, s.qkv_width, d), "b_qkv": (L, N, s.qkv_width),
        "w_proj": (L, N, d, d), "b_proj": (L, N, d),
        "ln2_g": (L, N, d), "ln2_b": (L, N, d),
        "w_up": (L, N, F, d), "b_up": (L, N, F),
        "w_down": (L, N, d, F), "b_down": (L, N, d),
        "w_concat": (d, N * d), "b_concat": (d,),
        "lnf_g": (d,), "lnf_b": (d,),
    }


# ----------------------------------------------------------------------------
# counter-based generator
# ----------------------------------------------------------------------------

def _mix32_scalar(x: int) -> int:
    """32-bit avalanche mix (xor-shift / odd-multiply rounds), pure Python."""
    x &= _M32
    x ^= x >> 16
    x = (x * 0x7FEB352D) & _M32
    x ^= x >> 15
    x = (x * 0x846CA68B) & _M32
    x ^= x >> 16
    return x


def _key_scalar(seed: int, tensor_id: int) -> int:
    return _mix32_scalar((seed * 0x9E3779B1 + tensor_id * 0x85EBCA77 + 0x01234567) & _M32)


def hash32_scalar(seed: int, tensor_id: int, index: int) -> int:
    """Reference scalar form of the generator: two mix rounds over the index."""
    key = _key_scalar(seed, tensor_id)
    lo, hi = index & _M32, index >> 32
    x = _mix32_scalar(lo ^ key)
    x = _mix32_scalar((x + hi * 0x27D4EB2F + tensor_id) & _M32)
    return x


def _mix32(x: torch.Tensor) -> torch.Tensor:
    # x: int64 holding values in [0, 2^32). Products wrap in 64 bits; the low
    # 32 bits are exact either way.
    x = x ^ (x >> 16)
    x = (x * 0x7FEB352D) & _M32
    x = x ^ (x >> 15)
    x = (x * 0x846CA68B) & _M32
    x = x ^ (x >> 16)
    return x


def hash32(seed: int, tensor_id: int, start: int, count: int, device) -> torch.Tensor:
    """hash32_scalar for indices start..start+count-1, as int64 in [0, 2^32)."""
    key = _key_scalar(seed, tensor_id)
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    lo, hi = idx & _M32, idx >> 32
    x = _mix32(lo ^ key)
    x = _mix32((x + hi * 0x27D4EB2F + tensor_id) & _M32)
    return x


_TABLE_CACHE: Dict[float, np.ndarray] = {}


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16 bit patterns (uint16). No NaN handling."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    return r


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def normal_table_bits(std: float) -> np.ndarray:
    """65536 bf16 bit patterns: std * Phi^-1((k + 1/2) / 65536), k = 0..65535.

    Drawing k uniformly gives a 16-bit-quantile discretisation of N(0, std^2),
    truncated at about 4.3 sigma.
    """
    if std not in _TABLE_CACHE:
        from scipy.special import ndtri
        k = np.arange(32768, 65536, dtype=np.float64)
        upper = f32_to_bf16_bits((ndtri((k + 0.5) / 65536.0) * std).astype(np.float32))
        # lower half mirrored (sign bit set) so the law is exactly symmetric
        _TABLE_CACHE[std] = np.concatenate([(upper | 0x8000)[::-1], upper]).astype(np.uint16)
    return _TABLE_CACHE[std]


def normal_bf16(seed: int, tensor_id: int, shape, std: float = 0.02, device="cpu",
                chunk: int = 1 << 24) -> torch.Tensor:
    """bf16 tensor of `shape`, element i = table[hash32(i) >> 16]."""
    n = int(np.prod(shape))
    table = torch.from_numpy(normal_table_bits(std).view(np.int16).copy()).to(device)
    out = torch.empty(n, dtype=torch.int16, device=device)
    for s in range(0, n, chunk):
        c = min(chunk, n - s)
        h = hash32(seed, tensor_id, s, c, device)
        out[s:s + c] = table[h >> 16]
    return out.view(torch.bfloat16).reshape(shape)


def uniform_tokens(seed: int, vocab: int, batch: int, seqlen: int, device="cpu") -> torch.Tensor:
    """int32 [batch, seqlen], uniform in [0, vocab)."""
    h = hash32(seed, TOKENS_TENSOR_ID, 0, batch * seqlen, device)
    return ((h * vocab) >> 32).to(torch.int32).reshape(batch, seqlen)


def normal_f16(seed: int, tensor_id: int, shape, std: float = 0.02, device="cpu") -> torch.Tensor:
    """The same draws as normal_bf16, held as IEEE half (every table value converts exactly except the few
    below 2^-14, which round to half's subnormal grid)."""
    return normal_bf16(seed, tensor_id, shape, std, device).to(torch.float16)


def make_weights(s: KrakenShape, seed: int = 0, device="cpu", std: float = 0.02,
                 bias: bool = True, dtype: str = "bf16") -> Dict[str, Optional[torch.Tensor]]:
    """All weight tensors of a Kraken model as 16-bit torch tensors (dtype "bf16" or "f16").

    Linear weights and (if bias) linear biases ~ N(0, std^2); LayerNorm gamma = 1,
    beta = 0.  With bias=False the bias entries are None (the ABI's NULL = zeros).
    """
    tdt = {"bf16": torch.bfloat16, "f16": torch.float16}[dtype]
    out: Dict[str, Optional[torch.Tensor]] = {}
    for tid, (name, shape) in enumerate(weight_shapes(s).items()):
        assert WEIGHT_FIELDS[tid] == name
        if name.endswith("_g") and name.startswith("ln"):
            out[name] = torch.ones(shape, dtype=tdt, device=device)
        elif name.endswith("_b") and name.startswith("ln"):
            out[name] = torch.zeros(shape, dtype=tdt, device=device)
        elif name.startswith("b_") and not bias:
            out[name] = None
        else:
            out[name] = normal_bf16(seed, tid, shape, std, device).to(tdt)
    return out


def bf16_tensor_to_bits(t: torch.Tensor) -> np.ndarray:
    """Host uint16 view of a 16-bit (bf16 or half) tensor (copied to CPU if needed)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def algorithmic_flops(s: KrakenShape, batch: Optional[int] = None, seqlen: Optional[int] = None,
                      last_positions_only: bool = False) -> Dict[str, float]:
    """FLOPs the prefill must perform: dense contractions, causal half of attention,
    last-position tail.  Masked attention work is not counted.
    last_positions_only: the count for a prefill that returns the logits of the last position of every sequence
    and therefore runs the last layer, past its qkv GEMM (the cache still needs every K and V row), on those B rows
    only: the last layer's output projection and FFN on the other T - B rows and its attention for every query but
    the last are not part of what has to be computed, and are not counted."""
    B = s.batch if batch is None else batch
    l = s.seqlen if seqlen is None else seqlen
    T = B * l
    N, L, d, F, H, hd, V = s.n_branch, s.n_layer, s.d_model, s.d_ff, s.n_head, s.head_dim, s.vocab
    gemm = 2.0 * T * N * L * (d * s.qkv_width + d * d + 2 * d * F)
    attn = float(N * L * B * H) * 4 * hd * (l * (l + 1) / 2)
    if last_positions_only:
        gemm -= 2.0 * (T - B) * N * (d * d + 2 * d * F)
        attn -= float(N * B * H) * 4 * hd * (l * (l + 1) / 2 - l)
    tail = 2.0 * B * (N * d * d + V * d)
    return {"gemm": gemm, "attn": attn, "tail": tail, "total": gemm + attn + tail}


def param_count(n_branch: int, n_layer: int, d_model: int, vocab: int, d_ff: int,
                max_pos: int = 0, with_concat: bool = False) -> int:
    """Weights of a Kraken model without biases and LayerNorms (Sec. 3.2 closed form):
    V*d + L*N*(4*d^2 + 2*d*d_ff), optionally plus learned positions and W_concat."""
    p = vocab * d_model + n_layer * n_branch * (4 * d_model * d_model + 2 * d_model * d_ff)
    if max_pos:
        p += max_pos * d_model
    if with_concat:
        p += n_branch * d_model * d_model
    return p
