"""Thin ctypes binding of libd3 (include/d3.h): argument marshalling only.

PyTorch supplies device memory and the CUDA stream; every step of the decode
path runs in the library's own kernels.  There is no fallback: if the library
cannot be loaded, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from . import build as _build

OK, EINVAL, ECAPACITY, ESTATE, ECUDA, ETIMEOUT = 0, -1, -2, -3, -4, -5
ANCHOR_START, ANCHOR_TAIL = 0, 1
FILL_NONE, FILL_COPY, FILL_RECOMPUTE = 0, 1, 2
MAX_BATCH, MAX_LAYERS, PROF_KINDS = 128, 128, 22
EXEC_AUTO, EXEC_KERNELS, EXEC_TENSOR, EXEC_FUSED = 0, 1, 2, 3
KV_CONTIGUOUS, KV_PAGED = 0, 1

EXPORTS = ("d3_depth", "d3_schedule", "d3_workspace_bytes", "d3_load", "d3_prefill",
           "d3_decode_step", "d3_decode_step_depths", "d3_depth_linear", "d3_saturation_probe",
           "d3_argmax", "d3_read_schedule", "d3_read_hidden", "d3_read_kv",
           "d3_set_exec", "d3_profile", "d3_read_profile", "d3_profile_name", "d3_read_fused_phases",
           "d3_decode_step_noalloc", "d3_noalloc_status", "d3_set_policy", "d3_set_wait_ns",
           "d3_stall_next_step", "d3_slot_pos",
           "d3_kv_pages_used", "d3_reset_slot", "d3_sync", "d3_free", "d3_strerror")


class Config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32)] + \
        [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim",
                                  "d_ffn", "vocab")] + \
        [("rms_eps", C.c_float), ("rope_base", C.c_float)] + \
        [(n, C.c_int32) for n in ("max_slots", "max_seq", "max_batch", "start_id", "anchor",
                                  "kv_fill", "kv_layout", "page_size", "n_pages")]


_PP = C.POINTER(C.c_void_p)


class Weights(C.Structure):
    _fields_ = [("embed_dev", C.c_void_p), ("lm_head_dev", C.c_void_p), ("final_norm_dev", C.c_void_p)] + \
        [(n, _PP) for n in ("attn_norm_dev", "wqkv_dev", "wo_dev", "mlp_norm_dev", "w_gate_dev",
                            "w_up_dev", "w_down_dev")]


class StepStats(C.Structure):
    _fields_ = [("n", C.POINTER(C.c_int32)), ("m_per_layer", C.POINTER(C.c_int32)),
                ("rows_layers", C.c_int64), ("layers_touched", C.c_int32),
                ("kernel_launches", C.c_int32), ("algorithmic_bytes", C.c_int64)]


class D3Error(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} ({code})")
        self.code = code


def _load() -> C.CDLL:
    path = _build.build()
    lib = C.CDLL(path)
    I32, I64, P = C.c_int32, C.c_int64, C.c_void_p
    lib.d3_depth.argtypes = [I32, C.c_double, I64]
    lib.d3_schedule.argtypes = [I32, C.c_double, I32, I32, I32] + [P] * 6 + [C.POINTER(I64), C.POINTER(I32)]
    lib.d3_workspace_bytes.argtypes = [C.POINTER(Config), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    lib.d3_load.argtypes = [C.POINTER(Config), C.POINTER(Weights), P, P, P, C.POINTER(P)]
    lib.d3_prefill.argtypes = [P, I32, P, I32, P]
    lib.d3_decode_step.argtypes = [P, I32, P, P, P, C.c_double, P, C.POINTER(StepStats), P]
    lib.d3_decode_step_depths.argtypes = [P, I32, P, P, P, P, C.POINTER(StepStats), P]
    lib.d3_depth_linear.argtypes = [I32, I32, I64, I64]
    lib.d3_saturation_probe.argtypes = [P, I32, P, P, P, P, P]
    lib.d3_argmax.argtypes = [P, P, I32, P]
    lib.d3_read_schedule.argtypes = [P, P, P, P, P]
    lib.d3_read_hidden.argtypes = [P, P]
    lib.d3_read_kv.argtypes = [P, I32, I32, I32, P, P]
    lib.d3_set_exec.argtypes = [P, I32]
    lib.d3_profile.argtypes = [P, I32]
    lib.d3_read_profile.argtypes = [P, P, P]
    lib.d3_read_fused_phases.argtypes = [P, P, P, P]
    lib.d3_profile_name.argtypes = [I32]
    lib.d3_profile_name.restype = C.c_char_p
    lib.d3_decode_step_noalloc.argtypes = [C.POINTER(Config), C.POINTER(Weights), P, I32, I32, I32, I32,
                                           C.c_double, P, P]
    lib.d3_noalloc_status.argtypes = [P]
    lib.d3_set_policy.argtypes = [P, I32, I32, I32]
    lib.d3_set_wait_ns.argtypes = [P, C.c_uint64]
    lib.d3_stall_next_step.argtypes = [P]
    lib.d3_slot_pos.argtypes = [P, I32]
    lib.d3_kv_pages_used.argtypes = [P]
    lib.d3_reset_slot.argtypes = [P, I32]
    lib.d3_sync.argtypes = [P]
    lib.d3_free.argtypes = [P]
    lib.d3_free.restype = None
    lib.d3_strerror.argtypes = [I32]
    lib.d3_strerror.restype = C.c_char_p
    return lib


LIB = _load()
LIB_PATH = _build.LIB


def strerror(code: int) -> str:
    return LIB.d3_strerror(code).decode()


def d3_depth(L: int, alpha: float, i: int) -> int:
    """floor(L * alpha^i); negative error code on bad arguments."""
    return int(LIB.d3_depth(L, alpha, i))


def d3_depth_linear(upper: int, lower: int, span: int, i: int) -> int:
    """upper - floor((upper - lower) * min(i, span) / span); negative error code on bad arguments."""
    return int(LIB.d3_depth_linear(upper, lower, span, i))


def d3_schedule(L: int, alpha: float, start_id: int, anchor: int, gen_index: Sequence[int]) -> Dict:
    """Host copy of the batch schedule (see include/d3.h)."""
    B = len(gen_index)
    gi = np.ascontiguousarray(np.asarray(gen_index, dtype=np.int32))
    n, lo, hi, perm = (np.zeros(max(B, 1), np.int32) for _ in range(4))
    m = np.zeros(max(L, 1), np.int32)
    rl, lt = C.c_int64(), C.c_int32()
    rc = LIB.d3_schedule(L, alpha, start_id, anchor, B, gi.ctypes.data, n.ctypes.data, lo.ctypes.data,
                         hi.ctypes.data, perm.ctypes.data, m.ctypes.data, C.byref(rl), C.byref(lt))
    if rc != OK:
        raise D3Error(rc, "d3_schedule")
    return {"n": n[:B], "lo": lo[:B], "hi": hi[:B], "perm": perm[:B], "m_per_layer": m[:L],
            "rows_layers": int(rl.value), "layers_touched": int(lt.value)}


def make_config(shape, max_slots: int, max_seq: int, max_batch: int, start_id: int = 0,
                anchor: int = ANCHOR_START, kv_fill: int = FILL_COPY, page_size: int = 0,
                n_pages: int = 0) -> Config:
    """page_size > 0 selects the paged KV layout with a pool of n_pages pages."""
    return Config(C.sizeof(Config), shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads,
                  shape.head_dim, shape.d_ffn, shape.vocab, shape.rms_eps, shape.rope_base,
                  max_slots, max_seq, max_batch, start_id, anchor, kv_fill,
                  KV_PAGED if page_size > 0 else KV_CONTIGUOUS, page_size, n_pages)


def d3_workspace_bytes(cfg: Config):
    kv, sc = C.c_size_t(), C.c_size_t()
    rc = LIB.d3_workspace_bytes(C.byref(cfg), C.byref(kv), C.byref(sc))
    if rc != OK:
        raise D3Error(rc, "d3_workspace_bytes")
    return int(kv.value), int(sc.value)


def _ptrs(tensors: List[torch.Tensor]):
    return (C.c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])


NOALLOC_SCRATCH_BYTES = 8 << 20


def d3_decode_step_noalloc(cfg: Config, weights: Dict[str, object], kv: torch.Tensor, slot: int, pos: int,
                           token: int, gen_index: int, alpha: float, logits: torch.Tensor,
                           stream: Optional[torch.cuda.Stream] = None) -> int:
    """One batch-1 decode step on the library's built-in scratch array (see
    include/d3.h).  Every tensor is the caller's; nothing is allocated here.
    Returns the library's status code instead of raising, so that callers can
    test the refusals."""
    arrays = {k: _ptrs(weights[k]) for k in ("attn_norm", "wqkv", "wo", "mlp_norm", "w_gate", "w_up",
                                             "w_down")}
    ws = Weights(weights["embed"].data_ptr(), weights["lm_head"].data_ptr(),
                 weights["final_norm"].data_ptr(),
                 *[C.cast(arrays[k], _PP) for k in ("attn_norm", "wqkv", "wo", "mlp_norm", "w_gate",
                                                    "w_up", "w_down")])
    st = stream if stream is not None else torch.cuda.current_stream(kv.device)
    return int(LIB.d3_decode_step_noalloc(C.byref(cfg), C.byref(ws), kv.data_ptr(), slot, pos, token,
                                          gen_index, float(alpha), logits.data_ptr(),
                                          C.c_void_p(st.cuda_stream)))


def d3_noalloc_status(stream: Optional[torch.cuda.Stream] = None) -> int:
    """Device status of the last d3_decode_step_noalloc on the current device (waits for the stream)."""
    st = stream if stream is not None else torch.cuda.current_stream()
    return int(LIB.d3_noalloc_status(C.c_void_p(st.cuda_stream)))


class D3Model:
    """A loaded model: owns the torch buffers the library borrows (weights given
    by the caller; KV cache and scratch allocated here with torch) and forwards
    each call to the C ABI."""

    def __init__(self, shape, weights: Dict[str, object], max_slots: int, max_seq: int,
                 max_batch: int = 1, start_id: int = 0, anchor: int = ANCHOR_START,
                 kv_fill: int = FILL_COPY, device="cuda:0", stream: Optional[torch.cuda.Stream] = None,
                 page_size: int = 0, n_pages: int = 0):
        self.shape = shape
        self.device = torch.device(device)
        self.cfg = make_config(shape, max_slots, max_seq, max_batch, start_id, anchor, kv_fill,
                               page_size, n_pages)
        kv_bytes, scratch_bytes = d3_workspace_bytes(self.cfg)
        self.kv_bytes, self.scratch_bytes = kv_bytes, scratch_bytes
        self.w = weights
        for k, v in weights.items():
            for t in (v if isinstance(v, list) else [v]):
                if t.device != self.device or t.dtype != torch.bfloat16 or not t.is_contiguous():
                    raise ValueError(f"weight {k}: expected contiguous bf16 on {self.device}")
        with torch.cuda.device(self.device):
            self.kv = torch.empty(kv_bytes, dtype=torch.uint8, device=self.device)
            self.scratch = torch.zeros(scratch_bytes, dtype=torch.uint8, device=self.device)
            self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
            self._arrays = {k: _ptrs(weights[k]) for k in ("attn_norm", "wqkv", "wo", "mlp_norm",
                                                           "w_gate", "w_up", "w_down")}
            ws = Weights(weights["embed"].data_ptr(), weights["lm_head"].data_ptr(),
                         weights["final_norm"].data_ptr(),
                         *[C.cast(self._arrays[k], _PP) for k in ("attn_norm", "wqkv", "wo", "mlp_norm",
                                                                  "w_gate", "w_up", "w_down")])
            h = C.c_void_p()
            rc = LIB.d3_load(C.byref(self.cfg), C.byref(ws), self.kv.data_ptr(), self.scratch.data_ptr(),
                             C.c_void_p(self.stream.cuda_stream), C.byref(h))
        if rc != OK:
            raise D3Error(rc, "d3_load")
        self.h = h

    def close(self):
        if getattr(self, "h", None) and LIB is not None:
            LIB.d3_free(self.h)
            self.h = None

    def __del__(self):
        self.close()

    def zero_kv(self):
        self.kv.zero_()

    def poison_kv(self):
        """Every cache entry := bf16 NaN, so that a read of an unwritten entry shows."""
        self.kv.view(torch.int16).fill_(0x7FC0)

    def d3_prefill(self, slot: int, tokens, logits: Optional[torch.Tensor] = None) -> torch.Tensor:
        t = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
        if logits is None:
            logits = torch.empty(self.shape.vocab, dtype=torch.float32, device=self.device)
        rc = LIB.d3_prefill(self.h, slot, t.ctypes.data, len(t), logits.data_ptr())
        if rc != OK:
            raise D3Error(rc, "d3_prefill")
        return logits

    def d3_decode_step_depths(self, slots, tokens, depths, logits: Optional[torch.Tensor] = None,
                              want_stats: bool = False, tokens_dev: Optional[torch.Tensor] = None):
        """d3_decode_step with the retained block count of every row given by the caller."""
        return self.d3_decode_step(slots, tokens, depths, None, logits, want_stats, tokens_dev)

    def d3_decode_step(self, slots, tokens, gen_index, alpha: Optional[float],
                       logits: Optional[torch.Tensor] = None, want_stats: bool = False,
                       tokens_dev: Optional[torch.Tensor] = None):
        """alpha None: `gen_index` holds retained block counts (d3_decode_step_depths)."""
        B = len(slots)
        s = np.ascontiguousarray(np.asarray(slots, dtype=np.int32))
        g = np.ascontiguousarray(np.asarray(gen_index, dtype=np.int32))
        t = None if tokens is None else np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
        if logits is None:
            logits = torch.empty((B, self.shape.vocab), dtype=torch.float32, device=self.device)
        st = None
        if want_stats:
            n = np.zeros(B, np.int32)
            m = np.zeros(self.shape.n_layers, np.int32)
            st = StepStats(n.ctypes.data_as(C.POINTER(C.c_int32)), m.ctypes.data_as(C.POINTER(C.c_int32)),
                           0, 0, 0, 0)
        if alpha is None:
            rc = LIB.d3_decode_step_depths(self.h, B, s.ctypes.data, None if t is None else t.ctypes.data,
                                           g.ctypes.data, logits.data_ptr(),
                                           C.byref(st) if st is not None else None,
                                           None if tokens_dev is None else tokens_dev.data_ptr())
        else:
            rc = LIB.d3_decode_step(self.h, B, s.ctypes.data, None if t is None else t.ctypes.data,
                                    g.ctypes.data, float(alpha), logits.data_ptr(),
                                    C.byref(st) if st is not None else None,
                                    None if tokens_dev is None else tokens_dev.data_ptr())
        if rc != OK:
            raise D3Error(rc, "d3_decode_step")
        if want_stats:
            return logits, {"n": n, "m_per_layer": m, "rows_layers": int(st.rows_layers),
                            "layers_touched": int(st.layers_touched),
                            "kernel_launches": int(st.kernel_launches),
                            "algorithmic_bytes": int(st.algorithmic_bytes)}
        return logits

    def d3_decode_one(self, slot: int, token: int, gen_index: int, alpha: float,
                      logits: torch.Tensor) -> torch.Tensor:
        """d3_decode_step for one row with the least marshalling (a greedy loop calls this once
        per token): the three one-element arrays are kept in the object, `logits` [vocab] or
        [1][vocab] is the caller's."""
        a = getattr(self, "_one", None)
        if a is None:
            a = self._one = ((C.c_int32 * 1)(), (C.c_int32 * 1)(), (C.c_int32 * 1)())
        a[0][0], a[1][0], a[2][0] = slot, token, gen_index
        rc = LIB.d3_decode_step(self.h, 1, a[0], a[1], a[2], float(alpha), logits.data_ptr(), None, None)
        if rc != OK:
            raise D3Error(rc, "d3_decode_step")
        return logits

    def d3_saturation_probe(self, slots, tokens):
        """One full-depth step; returns (logits [B][V], tokens [B][L] int32, conf [B][L] fp32),
        all on the device: what the LM head predicts from every block's output."""
        B, L = len(slots), self.shape.n_layers
        s = np.ascontiguousarray(np.asarray(slots, dtype=np.int32))
        t = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
        logits = torch.empty((B, self.shape.vocab), dtype=torch.float32, device=self.device)
        toks = torch.empty((B, L), dtype=torch.int32, device=self.device)
        conf = torch.empty((B, L), dtype=torch.float32, device=self.device)
        rc = LIB.d3_saturation_probe(self.h, B, s.ctypes.data, t.ctypes.data, logits.data_ptr(),
                                     toks.data_ptr(), conf.data_ptr())
        if rc != OK:
            raise D3Error(rc, "d3_saturation_probe")
        return logits, toks, conf

    def d3_argmax(self, logits: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        B = 1 if logits.dim() == 1 else logits.shape[0]
        if out is None:
            out = torch.empty(B, dtype=torch.int32, device=self.device)
        rc = LIB.d3_argmax(self.h, logits.data_ptr(), B, out.data_ptr())
        if rc != OK:
            raise D3Error(rc, "d3_argmax")
        return out

    def d3_read_schedule(self, B: int) -> Dict:
        n, perm = np.zeros(MAX_BATCH, np.int32), np.zeros(MAX_BATCH, np.int32)
        m = np.zeros(MAX_LAYERS, np.int32)
        cnt = np.zeros(2, np.int64)
        rc = LIB.d3_read_schedule(self.h, n.ctypes.data, perm.ctypes.data, m.ctypes.data, cnt.ctypes.data)
        if rc != OK:
            raise D3Error(rc, "d3_read_schedule")
        return {"n": n[:B], "perm": perm[:B], "m_per_layer": m[:self.shape.n_layers],
                "rows_layers": int(cnt[0]), "layers_touched": int(cnt[1])}

    def d3_read_hidden(self, B: int) -> np.ndarray:
        """Residual stream of the last step's rows (caller order).  The library writes as many
        rows as that step had (a prefill pass: up to max_batch), so the buffer is sized for the
        largest step; the first B rows are returned, or the LAST row when B == -1."""
        out = np.zeros((MAX_BATCH, self.shape.d_model), np.float32)
        rc = LIB.d3_read_hidden(self.h, out.ctypes.data)
        if rc != OK:
            raise D3Error(rc, "d3_read_hidden")
        return out[:B].copy()

    def d3_read_kv(self, layer: int, slot: int, pos: int):
        n = self.shape.n_kv_heads * self.shape.head_dim
        k, v = np.zeros(n, np.float32), np.zeros(n, np.float32)
        rc = LIB.d3_read_kv(self.h, layer, slot, pos, k.ctypes.data, v.ctypes.data)
        if rc != OK:
            raise D3Error(rc, "d3_read_kv")
        return k, v

    def d3_set_exec(self, mode: int) -> None:
        rc = LIB.d3_set_exec(self.h, mode)
        if rc != OK:
            raise D3Error(rc, "d3_set_exec")

    def d3_profile(self, enable: bool) -> None:
        rc = LIB.d3_profile(self.h, int(enable))
        if rc != OK:
            raise D3Error(rc, "d3_profile")

    def d3_read_profile(self) -> Dict[str, Dict[str, float]]:
        """{kernel class: {"ms": total device ms, "launches": count}} since the last read."""
        ms = np.zeros(PROF_KINDS, np.float32)
        cnt = np.zeros(PROF_KINDS, np.int32)
        rc = LIB.d3_read_profile(self.h, ms.ctypes.data, cnt.ctypes.data)
        if rc != OK:
            raise D3Error(rc, "d3_read_profile")
        return {LIB.d3_profile_name(k).decode(): {"ms": float(ms[k]), "launches": int(cnt[k])}
                for k in range(PROF_KINDS) if cnt[k] > 0}

    def d3_read_fused_phases(self) -> np.ndarray:
        """Per-CTA cycle counters of the single-kernel step's phases, [ctas][phases] (not cleared)."""
        buf = np.zeros((192, 16), np.int64)
        nc, nph = C.c_int32(), C.c_int32()
        rc = LIB.d3_read_fused_phases(self.h, buf.ctypes.data, C.byref(nc), C.byref(nph))
        if rc != OK:
            raise D3Error(rc, "d3_read_fused_phases")
        return buf.reshape(-1)[:nc.value * nph.value].reshape(nc.value, nph.value).copy()

    def d3_slot_pos(self, slot: int) -> int:
        return int(LIB.d3_slot_pos(self.h, slot))

    def d3_kv_pages_used(self) -> int:
        rc = int(LIB.d3_kv_pages_used(self.h))
        if rc < 0:
            raise D3Error(rc, "d3_kv_pages_used")
        return rc

    def d3_reset_slot(self, slot: int) -> None:
        rc = LIB.d3_reset_slot(self.h, slot)
        if rc != OK:
            raise D3Error(rc, "d3_reset_slot")

    def d3_sync(self) -> None:
        rc = LIB.d3_sync(self.h)
        if rc != OK:
            raise D3Error(rc, "d3_sync")

    def d3_set_policy(self, start_id: int, anchor: int, kv_fill: int) -> None:
        rc = LIB.d3_set_policy(self.h, start_id, anchor, kv_fill)
        if rc != OK:
            raise D3Error(rc, "d3_set_policy")

    def d3_set_wait_ns(self, ns: int) -> None:
        rc = LIB.d3_set_wait_ns(self.h, int(ns))
        if rc != OK:
            raise D3Error(rc, "d3_set_wait_ns")

    def d3_stall_next_step(self) -> None:
        rc = LIB.d3_stall_next_step(self.h)
        if rc != OK:
            raise D3Error(rc, "d3_stall_next_step")
