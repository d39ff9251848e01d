"""CPU oracle of D3 decoding: TEST INFRASTRUCTURE, not a product path.

Builds `d3_oracle.c` with gcc into two shared objects (fp64 arithmetic, and
fp32 for comparison) and wraps them with ctypes.  Only the tests, the smoke
check and the CPU-baseline timing import this package; the CUDA library and
its Python binding never do.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "d3_oracle.c")
_LIBS = {"f64": os.path.join(_HERE, "libd3oracle.so"),
         "f32": os.path.join(_HERE, "libd3oracle_f32.so")}

ANCHOR_START, ANCHOR_TAIL = 0, 1
FILL_NONE, FILL_COPY, FILL_RECOMPUTE = 0, 1, 2


def build(force: bool = False) -> None:
    """Compile the oracle (gcc, -O2, OpenMP) if the objects are missing or stale."""
    for kind, lib in _LIBS.items():
        if not force and os.path.exists(lib) and os.path.getmtime(lib) >= os.path.getmtime(_SRC):
            continue
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-Wall",
               "-DD3O_REAL=" + ("double" if kind == "f64" else "float"),
               _SRC, "-o", lib, "-lm"]
        subprocess.run(cmd, check=True)


class _Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab")] + \
               [("rms_eps", C.c_double), ("rope_base", C.c_double)] + \
               [(n, C.c_int32) for n in
                ("max_slots", "max_seq", "start_id", "anchor", "kv_fill", "kv_round_bf16")]


_PP = C.POINTER(C.c_void_p)


class _Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p)] + \
               [(n, _PP) for n in ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm",
                                   "w_gate", "w_up", "w_down")]


_loaded: Dict[str, C.CDLL] = {}


def _lib(kind: str) -> C.CDLL:
    lib = _loaded.get(kind)
    if lib is None:
        build()
        lib = C.CDLL(_LIBS[kind])
        lib.d3o_create.restype = C.c_void_p
        lib.d3o_create.argtypes = [C.POINTER(_Config), C.POINTER(_Weights)]
        lib.d3o_destroy.argtypes = [C.c_void_p]
        lib.d3o_poison_kv.argtypes = [C.c_void_p]
        lib.d3o_set_policy.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32]
        lib.d3o_slot_pos.argtypes = [C.c_void_p, C.c_int32]
        lib.d3o_depth.argtypes = [C.c_int32, C.c_double, C.c_int64]
        lib.d3o_depth_pow.argtypes = [C.c_int32, C.c_double, C.c_int64]
        lib.d3o_window.argtypes = [C.c_int32, C.c_double, C.c_int64, C.c_int32, C.c_int32,
                                   C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        lib.d3o_schedule.argtypes = [C.c_int32, C.c_double, C.c_int32, C.c_int32, C.c_int32] + \
            [C.c_void_p] * 6 + [C.POINTER(C.c_int64), C.POINTER(C.c_int32)]
        lib.d3o_prefill.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p,
                                    C.c_void_p]
        lib.d3o_decode_step.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_double, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.d3o_decode_step_depths.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                               C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.d3o_depth_linear.argtypes = [C.c_int32, C.c_int32, C.c_int64, C.c_int64]
        lib.d3o_probe.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(C.c_int32),
                                  C.POINTER(C.c_double)]
        lib.d3o_window_of_depth.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                            C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        lib.d3o_decode_layers.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int32,
                                          C.c_void_p, C.c_void_p]
        lib.d3o_forward_nocache.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        lib.d3o_read_kv.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                    C.c_void_p]
        lib.d3o_argmax.argtypes = [C.c_void_p, C.c_int32]
        _loaded[kind] = lib
    return lib


def threads() -> int:
    """Threads the oracle's matrix-vector products use."""
    return int(_lib("f64").d3o_threads())


def depth(L: int, alpha: float, i: int) -> int:
    """floor(L * alpha^i), by repeated multiplication."""
    return int(_lib("f64").d3o_depth(L, alpha, i))


def depth_pow(L: int, alpha: float, i: int) -> int:
    return int(_lib("f64").d3o_depth_pow(L, alpha, i))


def depth_linear(upper: int, lower: int, span: int, i: int) -> int:
    """Linear decay from `upper` layers at i = 0 to `lower` at i = span, constant after."""
    return int(_lib("f64").d3o_depth_linear(upper, lower, span, i))


def window_of_depth(L: int, n: int, start_id: int, anchor: int = ANCHOR_START):
    """(retained count, lo, hi) for a retained count given by the caller."""
    lo, hi = C.c_int32(), C.c_int32()
    r = _lib("f64").d3o_window_of_depth(L, n, start_id, anchor, C.byref(lo), C.byref(hi))
    return int(r), int(lo.value), int(hi.value)


def window(L: int, alpha: float, i: int, start_id: int, anchor: int = ANCHOR_START):
    """(retained count, lo, hi) with [lo, hi) the dropped layers of T_i."""
    lo, hi = C.c_int32(), C.c_int32()
    n = _lib("f64").d3o_window(L, alpha, i, start_id, anchor, C.byref(lo), C.byref(hi))
    return int(n), int(lo.value), int(hi.value)


def schedule(L: int, alpha: float, start_id: int, anchor: int, gen_index: Sequence[int]):
    """Batch schedule: dict with n, lo, hi, perm, m_per_layer, rows_layers, layers_touched."""
    B = len(gen_index)
    gi = np.asarray(gen_index, dtype=np.int32)
    n, lo, hi, perm = (np.zeros(B, np.int32) for _ in range(4))
    m = np.zeros(L, np.int32)
    rl, lt = C.c_int64(), C.c_int32()
    rc = _lib("f64").d3o_schedule(L, alpha, start_id, anchor, B, gi.ctypes.data, n.ctypes.data,
                                  lo.ctypes.data, hi.ctypes.data, perm.ctypes.data,
                                  m.ctypes.data, C.byref(rl), C.byref(lt))
    if rc != 0:
        raise ValueError("invalid schedule arguments")
    return {"n": n, "lo": lo, "hi": hi, "perm": perm, "m_per_layer": m,
            "rows_layers": int(rl.value), "layers_touched": int(lt.value)}


def _ptr_array(tensors: List[torch.Tensor]):
    arr = (C.c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])
    return arr


class Oracle:
    """One model instance of the CPU oracle.

    `weights` is the dictionary `inputs.make_weights` returns (CPU bf16
    tensors); the oracle borrows their storage, so this object keeps them alive.
    """

    def __init__(self, shape, weights, max_slots: int, max_seq: int, start_id: int = 0,
                 anchor: int = ANCHOR_START, kv_fill: int = FILL_COPY,
                 kv_round_bf16: bool = False, real: str = "f64"):
        self.lib = _lib(real)
        self.shape = shape
        self.w = weights
        for k, v in weights.items():
            for t in (v if isinstance(v, list) else [v]):
                assert t.device.type == "cpu" and t.dtype == torch.bfloat16 and t.is_contiguous(), k
        nq = shape.n_q_heads * shape.head_dim
        nkv = shape.n_kv_heads * shape.head_dim
        self._wq = [w[:nq] for w in weights["wqkv"]]
        self._wk = [w[nq:nq + nkv] for w in weights["wqkv"]]
        self._wv = [w[nq + nkv:] for w in weights["wqkv"]]
        cfg = _Config(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads,
                      shape.head_dim, shape.d_ffn, shape.vocab, shape.rms_eps, shape.rope_base,
                      max_slots, max_seq, start_id, anchor, kv_fill, int(kv_round_bf16))
        self._arrays = {
            "attn_norm": _ptr_array(weights["attn_norm"]), "wq": _ptr_array(self._wq),
            "wk": _ptr_array(self._wk), "wv": _ptr_array(self._wv),
            "wo": _ptr_array(weights["wo"]), "mlp_norm": _ptr_array(weights["mlp_norm"]),
            "w_gate": _ptr_array(weights["w_gate"]), "w_up": _ptr_array(weights["w_up"]),
            "w_down": _ptr_array(weights["w_down"]),
        }
        ws = _Weights(weights["embed"].data_ptr(), weights["lm_head"].data_ptr(),
                      weights["final_norm"].data_ptr(),
                      *[C.cast(self._arrays[n], _PP) for n in
                        ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up",
                         "w_down")])
        self.h = self.lib.d3o_create(C.byref(cfg), C.byref(ws))
        if not self.h:
            raise ValueError("oracle rejected the configuration")

    def close(self):
        if getattr(self, "h", None):
            self.lib.d3o_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()

    def poison_kv(self):
        self.lib.d3o_poison_kv(self.h)

    def set_policy(self, start_id: int, anchor: int, kv_fill: int):
        self.lib.d3o_set_policy(self.h, start_id, anchor, kv_fill)

    def slot_pos(self, slot: int) -> int:
        return int(self.lib.d3o_slot_pos(self.h, slot))

    def prefill(self, slot: int, tokens, want_hidden: bool = False):
        """All prompt tokens through all layers; returns logits [vocab] (and hidden [d])."""
        t = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
        logits = np.zeros(self.shape.vocab, np.float64)
        hidden = np.zeros(self.shape.d_model, np.float64)
        rc = self.lib.d3o_prefill(self.h, slot, t.ctypes.data, len(t), logits.ctypes.data,
                                  hidden.ctypes.data)
        if rc != 0:
            raise ValueError(f"oracle prefill failed ({rc})")
        return (logits, hidden) if want_hidden else logits

    def decode_step(self, slots, tokens, gen_index, alpha: float, want_trace: bool = False):
        """One generation step; returns dict(logits [B][V], hidden [B][d], trace?)."""
        B = len(slots)
        s = np.ascontiguousarray(np.asarray(slots, dtype=np.int32))
        t = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
        g = np.ascontiguousarray(np.asarray(gen_index, dtype=np.int32))
        logits = np.zeros((B, self.shape.vocab), np.float64)
        hidden = np.zeros((B, self.shape.d_model), np.float64)
        trace = np.zeros((B, self.shape.n_layers + 1, self.shape.d_model), np.float64) \
            if want_trace else None
        rc = self.lib.d3o_decode_step(self.h, B, s.ctypes.data, t.ctypes.data, g.ctypes.data,
                                      float(alpha), logits.ctypes.data, hidden.ctypes.data,
                                      trace.ctypes.data if want_trace else None)
        if rc != 0:
            raise ValueError(f"oracle decode_step failed ({rc})")
        out = {"logits": logits, "hidden": hidden}
        if want_trace:
            out["trace"] = trace
        return out

    def decode_step_depths(self, slots, tokens, depths):
        """One generation step with the retained count of every row given by the caller."""
        B = len(slots)
        s = np.ascontiguousarray(np.asarray(slots, dtype=np.int32))
        t = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
        n = np.ascontiguousarray(np.asarray(depths, dtype=np.int32))
        logits = np.zeros((B, self.shape.vocab), np.float64)
        hidden = np.zeros((B, self.shape.d_model), np.float64)
        rc = self.lib.d3o_decode_step_depths(self.h, B, s.ctypes.data, t.ctypes.data, n.ctypes.data,
                                             logits.ctypes.data, hidden.ctypes.data, None)
        if rc != 0:
            raise ValueError(f"oracle decode_step_depths failed ({rc})")
        return {"logits": logits, "hidden": hidden}

    def probe(self, hidden):
        """(token, confidence, logits) that lm_head(final_norm(hidden)) predicts."""
        h = np.ascontiguousarray(np.asarray(hidden, dtype=np.float64))
        logits = np.zeros(self.shape.vocab, np.float64)
        tok, conf = C.c_int32(), C.c_double()
        self.lib.d3o_probe(self.h, h.ctypes.data, logits.ctypes.data, C.byref(tok), C.byref(conf))
        return int(tok.value), float(conf.value), logits

    def saturation_probe(self, slots, tokens):
        """One full-depth step; per row and block i = 1..L the token and confidence that
        lm_head(h^i) predicts.  Returns dict(logits, hidden, tokens [B][L], conf [B][L])."""
        L = self.shape.n_layers
        r = self.decode_step(slots, tokens, [1] * len(slots), 1.0, want_trace=True)
        toks = np.zeros((len(slots), L), np.int32)
        conf = np.zeros((len(slots), L), np.float64)
        for b in range(len(slots)):
            for i in range(1, L + 1):
                toks[b, i - 1], conf[b, i - 1], _ = self.probe(r["trace"][b, i])
        r["tokens"], r["conf"] = toks, conf
        return r

    def decode_layers(self, slot: int, token: int, layers: Sequence[int]):
        """One step over exactly the listed blocks (no schedule, no fill)."""
        ls = np.ascontiguousarray(np.asarray(layers, dtype=np.int32))
        logits = np.zeros(self.shape.vocab, np.float64)
        hidden = np.zeros(self.shape.d_model, np.float64)
        rc = self.lib.d3o_decode_layers(self.h, slot, token, ls.ctypes.data, len(ls),
                                        logits.ctypes.data, hidden.ctypes.data)
        if rc != 0:
            raise ValueError(f"oracle decode_layers failed ({rc})")
        return logits, hidden

    def forward_nocache(self, tokens):
        """Full-depth logits of every position, recomputed without a cache."""
        t = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
        logits = np.zeros((len(t), self.shape.vocab), np.float64)
        rc = self.lib.d3o_forward_nocache(self.h, t.ctypes.data, len(t), logits.ctypes.data)
        if rc != 0:
            raise ValueError("oracle forward_nocache failed")
        return logits

    def read_kv(self, layer: int, slot: int, t: int):
        n = self.shape.n_kv_heads * self.shape.head_dim
        k, v = np.zeros(n, np.float64), np.zeros(n, np.float64)
        self.lib.d3o_read_kv(self.h, layer, slot, t, k.ctypes.data, v.ctypes.data)
        return k, v


def argmax(v: np.ndarray) -> int:
    """Lowest index of the maximum."""
    v = np.ascontiguousarray(v, dtype=np.float64)
    return int(_lib("f64").d3o_argmax(v.ctypes.data, v.size))


def _real_array(lib, values) -> np.ndarray:
    dt = np.float64 if lib.d3o_real_bytes() == 8 else np.float32
    return np.ascontiguousarray(np.asarray(values, dtype=dt))


def rmsnorm(x, gain_bf16: torch.Tensor, eps: float, real: str = "f64") -> np.ndarray:
    lib = _lib(real)
    xa = _real_array(lib, x)
    out = np.zeros_like(xa)
    lib.d3o_rmsnorm.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_double, C.c_void_p]
    lib.d3o_rmsnorm(xa.ctypes.data, gain_bf16.data_ptr(), xa.size, eps, out.ctypes.data)
    return out.astype(np.float64)


def rope(v, pos: int, base: float, real: str = "f64") -> np.ndarray:
    lib = _lib(real)
    va = _real_array(lib, v).copy()
    lib.d3o_rope.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_double]
    lib.d3o_rope(va.ctypes.data, va.size, pos, base)
    return va.astype(np.float64)


def round_bf16(x, real: str = "f64") -> np.ndarray:
    """The bf16 value nearest to each element (ties to even), as the oracle stores K and V
    when `kv_round_bf16` is set."""
    lib = _lib(real)
    xa = _real_array(lib, x).ravel()
    out = np.zeros_like(xa)
    lib.d3o_round_bf16.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
    lib.d3o_round_bf16(xa.ctypes.data, xa.size, out.ctypes.data)
    return out.astype(np.float64)


def softmax(s, real: str = "f64") -> np.ndarray:
    lib = _lib(real)
    sa = _real_array(lib, s).copy()
    lib.d3o_softmax.argtypes = [C.c_void_p, C.c_int32]
    lib.d3o_softmax(sa.ctypes.data, sa.size)
    return sa.astype(np.float64)
