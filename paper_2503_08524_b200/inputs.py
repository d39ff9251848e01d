"""Seeded synthetic inputs: model shapes, weights and token ids.

This module serves both the CUDA library's callers and the CPU oracle's tests.
It holds no arithmetic of the decoding method itself: only shapes, a
counter-based integer hash, and a table lookup that turns hash bits into
bf16 values with a normal distribution.

Every value is a pure function of (seed, stream id, element index), computed
with integer tensor operations only, so the same call gives bit-identical
tensors on the CPU and on a GPU:

    h      = mix64(key(seed, stream) + index * GOLDEN)      (a splitmix64-style finaliser)
    weight = TABLE[h >> 48]     TABLE[j] = bf16( std * Phi^-1((j + 0.5) / 65536) )
    token  = (h >> 11) mod vocab

The weights stand in for the Llama-2 checkpoints the paper evaluates (random
init N(0, 0.02), norm gains 1.0); the token ids stand in for its tokenised
prompts (uniform over the vocabulary).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List

import torch

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB


def _s64(v: int) -> int:
    """Two's-complement view of an unsigned 64-bit constant."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def _lsr(x: torch.Tensor, n: int) -> torch.Tensor:
    """Logical right shift of int64 lanes."""
    return (x >> n) & ((1 << (64 - n)) - 1)


def _mix64(x: torch.Tensor) -> torch.Tensor:
    x = (x ^ _lsr(x, 30)) * _s64(_M1)
    x = (x ^ _lsr(x, 27)) * _s64(_M2)
    return x ^ _lsr(x, 31)


def _key(seed: int, stream: int) -> int:
    """Scalar key for one (seed, stream) pair, mixed on the host with Python ints."""
    x = (seed * _GOLDEN + stream * _M1 + 0x632BE59BD9B4E019) & _MASK64
    x = ((x ^ (x >> 30)) * _M1) & _MASK64
    x = ((x ^ (x >> 27)) * _M2) & _MASK64
    return x ^ (x >> 31)


def hash_bits(seed: int, stream: int, start: int, count: int, device) -> torch.Tensor:
    """int64 tensor of `count` hashed 64-bit words for indices start .. start+count-1."""
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    return _mix64(idx * _s64(_GOLDEN) + _s64(_key(seed, stream)))


_TABLES: Dict[float, torch.Tensor] = {}


def normal_table(std: float) -> torch.Tensor:
    """65536 bf16 quantiles of N(0, std^2), built once on the CPU in fp64."""
    t = _TABLES.get(std)
    if t is None:
        p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
        z = math.sqrt(2.0) * torch.erfinv(2.0 * p - 1.0)
        t = (z * std).to(torch.float32).to(torch.bfloat16)
        _TABLES[std] = t
    return t


def normal_bf16(seed: int, stream: int, shape, device="cpu", std: float = 0.02) -> torch.Tensor:
    """bf16 tensor of the given shape with N(0, std^2) entries."""
    n = 1
    for s in shape:
        n *= int(s)
    table = normal_table(std).to(device)
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    chunk = 1 << 26
    for a in range(0, n, chunk):
        c = min(chunk, n - a)
        h = hash_bits(seed, stream, a, c, device)
        out[a:a + c] = table[_lsr(h, 48)]
    return out.view(*shape)


def token_ids(seed: int, stream: int, count: int, vocab: int, device="cpu") -> torch.Tensor:
    """int32 token ids uniform over [0, vocab)."""
    h = hash_bits(seed, stream, 0, count, device)
    return (_lsr(h, 11) % vocab).to(torch.int32)


def uniform_ints(seed: int, stream: int, count: int, lo: int, hi: int) -> List[int]:
    """`count` integers uniform over [lo, hi] (inclusive), as Python ints."""
    h = hash_bits(seed, stream, 0, count, "cpu")
    return [int(v) for v in (_lsr(h, 11) % (hi - lo + 1) + lo)]


@dataclasses.dataclass(frozen=True)
class ModelShape:
    """Sizes of a Llama-style decoder."""
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rms_eps: float = 1e-5
    rope_base: float = 10000.0

    @property
    def qkv_rows(self) -> int:
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim

    @property
    def layer_weight_bytes(self) -> int:
        d, f = self.d_model, self.d_ffn
        return 2 * (self.qkv_rows * d + d * self.n_q_heads * self.head_dim + 3 * d * f + 2 * d)

    @property
    def head_weight_bytes(self) -> int:
        return 2 * (self.vocab * self.d_model + self.d_model)

    @property
    def kv_bytes_per_token_layer(self) -> int:
        return 2 * self.n_kv_heads * self.head_dim * 2

    def with_layers(self, n_layers: int) -> "ModelShape":
        return dataclasses.replace(self, n_layers=n_layers, name=f"{self.name}-L{n_layers}")


TINY = ModelShape("tiny", 4, 256, 4, 4, 64, 688, 1024)
TINY_GQA = ModelShape("tiny-gqa", 4, 256, 8, 2, 32, 688, 1024)
LLAMA_7B = ModelShape("llama2-7b-shape", 32, 4096, 32, 32, 128, 11008, 32000)
LLAMA_13B = ModelShape("llama2-13b-shape", 40, 5120, 40, 40, 128, 13824, 32000)
LLAMA_70B = ModelShape("llama2-70b-shape", 80, 8192, 64, 8, 128, 28672, 32000)

BASE_SEED = 250308524

# stream ids of the tensors of one model
_S_EMBED, _S_HEAD, _S_LAYER0, _S_PER_LAYER = 1, 2, 16, 8
_S_TOKENS = 1 << 20


def make_weights(shape: ModelShape, seed: int, device="cpu", std: float = 0.02,
                 gain_jitter: float = 0.0) -> Dict[str, object]:
    """Random-init weights of `shape`: linear and embedding matrices N(0, std^2)
    in bf16, row-major [out][in]; norm gains 1.0 (+ N(0, gain_jitter^2) when a
    test wants gains that matter).  Q, K and V of a layer are the row blocks of
    one fused matrix `wqkv` ([Hq*dh | Hkv*dh | Hkv*dh] rows)."""
    d, f = shape.d_model, shape.d_ffn
    gain_stream = [1 << 16]

    def ones():
        g = torch.ones(d, dtype=torch.bfloat16, device=device)
        if gain_jitter > 0.0:
            gain_stream[0] += 1
            j = normal_bf16(seed, gain_stream[0], (d,), device, gain_jitter)
            g = (g.float() + j.float()).to(torch.bfloat16)
        return g
    w: Dict[str, object] = {
        "embed": normal_bf16(seed, _S_EMBED, (shape.vocab, d), device, std),
        "lm_head": normal_bf16(seed, _S_HEAD, (shape.vocab, d), device, std),
        "final_norm": ones(),
        "attn_norm": [], "wqkv": [], "wo": [], "mlp_norm": [],
        "w_gate": [], "w_up": [], "w_down": [],
    }
    for l in range(shape.n_layers):
        s = _S_LAYER0 + l * _S_PER_LAYER
        w["attn_norm"].append(ones())
        w["wqkv"].append(normal_bf16(seed, s + 0, (shape.qkv_rows, d), device, std))
        w["wo"].append(normal_bf16(seed, s + 1, (d, shape.n_q_heads * shape.head_dim), device, std))
        w["mlp_norm"].append(ones())
        w["w_gate"].append(normal_bf16(seed, s + 2, (f, d), device, std))
        w["w_up"].append(normal_bf16(seed, s + 3, (f, d), device, std))
        w["w_down"].append(normal_bf16(seed, s + 4, (d, f), device, std))
    return w


def weights_to(w: Dict[str, object], device) -> Dict[str, object]:
    """The same weights on another device."""
    out: Dict[str, object] = {}
    for k, v in w.items():
        out[k] = [t.to(device) for t in v] if isinstance(v, list) else v.to(device)
    return out


def prompt_tokens(shape: ModelShape, seed: int, row: int, length: int) -> torch.Tensor:
    """Prompt of `length` uniform-random token ids for batch row `row` (CPU int32)."""
    return token_ids(seed, _S_TOKENS + row, length, shape.vocab, "cpu")
