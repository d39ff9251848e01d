"""Host side of the C ABI (no GPU): the library loads, exports what the header
declares, validates arguments, and its host schedule equals the oracle's."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle as O
from paper_2503_08524_b200 import binding as B
from paper_2503_08524_b200 import inputs as I

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "d3.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(d3_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(B.LIB, n), n
    assert set(names) == set(B.EXPORTS)
    assert os.path.exists(B.LIB_PATH)


@pytest.mark.parametrize("L,alpha", [(4, 0.98), (4, 0.95), (32, 0.999), (32, 0.995), (32, 0.997),
                                     (40, 0.998), (80, 0.998), (32, 0.9), (80, 0.9999), (32, 1.0)])
def test_depth_equals_oracle(L, alpha):
    for i in list(range(0, 600)) + [1023, 5000, 100000]:
        assert B.d3_depth(L, alpha, i) == O.depth(L, alpha, i)


def test_depth_margin_from_integers():
    # floor() is safe: L*alpha^i stays well away from an integer boundary (fp64 error ~1e-13)
    import math
    from fractions import Fraction
    for L, alpha in [(4, 0.98), (4, 0.95), (32, 0.999), (32, 0.995), (32, 0.997), (40, 0.998), (80, 0.998)]:
        worst = 1.0
        for i in range(1, 1300):
            v = L * Fraction(alpha) ** i
            if v < 0.5:
                break                      # depth 0 from here on: no boundary left to cross
            frac = float(v - math.floor(v))
            worst = min(worst, frac, 1 - frac)
        assert worst > 1e-9, (L, alpha, worst)


def test_depth_rejects_bad_arguments():
    for bad in (0.0, -1.0, 1.5, float("nan"), float("inf")):
        assert B.d3_depth(32, bad, 1) == B.EINVAL
    assert B.d3_depth(32, 0.9, -1) == B.EINVAL and B.d3_depth(-1, 0.9, 1) == B.EINVAL


@pytest.mark.parametrize("anchor", [B.ANCHOR_START, B.ANCHOR_TAIL])
def test_host_schedule_equals_oracle(anchor):
    rng = np.random.default_rng(11)
    for L, alpha, s in [(32, 0.997, 6), (4, 0.95, 0), (4, 0.98, 1), (40, 0.998, 8), (80, 0.998, 16),
                        (32, 0.9, 19), (128, 0.99, 30), (32, 1.0, 6)]:
        for Bn in (1, 2, 5, 32, 64):
            gi = rng.integers(1, 700, size=Bn).astype(np.int32)
            gi[Bn // 2] = gi[0]
            a = B.d3_schedule(L, alpha, s, anchor, gi)
            o = O.schedule(L, alpha, s, anchor, gi)
            for k in ("n", "lo", "hi", "perm", "m_per_layer"):
                assert np.array_equal(a[k], o[k]), (k, L, alpha, s, Bn)
            assert a["rows_layers"] == o["rows_layers"] and a["layers_touched"] == o["layers_touched"]


def test_schedule_rejects_bad_arguments():
    for kw in [dict(L=0), dict(L=129), dict(alpha=0.0), dict(alpha=float("nan")), dict(start_id=33),
               dict(start_id=-1), dict(anchor=2), dict(gen_index=[-1]), dict(gen_index=[1] * 129)]:
        args = dict(L=32, alpha=0.9, start_id=6, anchor=0, gen_index=[1, 2])
        args.update(kw)
        with pytest.raises(B.D3Error) as e:
            B.d3_schedule(**args)
        assert e.value.code == B.EINVAL


def test_workspace_and_load_validation():
    cfg = B.make_config(I.LLAMA_7B, max_slots=1, max_seq=1024, max_batch=1)
    kv, scratch = B.d3_workspace_bytes(cfg)
    assert kv == 2 * 32 * 1 * 32 * 1024 * 128 * 2
    assert scratch > 0 and scratch % 256 == 0
    for field, bad in [("struct_size", 4), ("n_layers", 0), ("n_layers", 129), ("d_model", 4100),
                       ("head_dim", 96), ("n_kv_heads", 5), ("max_batch", 129), ("start_id", 33),
                       ("anchor", 7), ("kv_fill", 3), ("kv_layout", 1), ("d_ffn", 11009)]:
        c = B.make_config(I.LLAMA_7B, 1, 1024, 1)
        setattr(c, field, bad)
        with pytest.raises(B.D3Error) as e:
            B.d3_workspace_bytes(c)
        assert e.value.code == B.EINVAL, field
    # paged layout: pool of n_pages pages of page_size positions, one block each
    pc = B.make_config(I.LLAMA_7B, 4, 1024, 4, page_size=64, n_pages=100)
    pkv, pscratch = B.d3_workspace_bytes(pc)
    assert pkv == 2 * 100 * 32 * 64 * 128 * 2
    assert pscratch > B.d3_workspace_bytes(B.make_config(I.LLAMA_7B, 4, 1024, 4))[1]   # + the page table
    for field, bad in [("page_size", 48), ("page_size", 8), ("page_size", 2048), ("n_pages", 1),
                       ("max_seq", 1000), ("kv_layout", 0)]:
        c = B.make_config(I.LLAMA_7B, 4, 1024, 4, page_size=64, n_pages=100)
        setattr(c, field, bad)
        with pytest.raises(B.D3Error) as e:
            B.d3_workspace_bytes(c)
        assert e.value.code == B.EINVAL, field
    h = C.c_void_p()
    assert B.LIB.d3_load(C.byref(cfg), None, None, None, None, C.byref(h)) == B.EINVAL
    assert B.LIB.d3_load(None, None, None, None, None, C.byref(h)) == B.EINVAL
    # null model handles never reach a launch
    assert B.LIB.d3_prefill(None, 0, None, 1, None) == B.EINVAL
    assert B.LIB.d3_decode_step(None, 1, None, None, None, 0.9, None, None, None) == B.EINVAL
    assert B.LIB.d3_sync(None) == B.EINVAL and B.LIB.d3_slot_pos(None, 0) == B.EINVAL
    assert B.LIB.d3_set_policy(None, 0, 0, 0) == B.EINVAL and B.LIB.d3_set_wait_ns(None, 5) == B.EINVAL
    assert B.LIB.d3_stall_next_step(None) == B.EINVAL
    assert B.strerror(B.ESTATE) != B.strerror(B.ECAPACITY)
    assert B.strerror(-99) == "unknown error"


def test_linear_depth_matches_the_oracle_rule():
    for upper, lower, span in [(32, 8, 255), (40, 14, 512), (80, 48, 100), (4, 0, 3), (7, 7, 10)]:
        for i in list(range(0, span + 5, max(1, span // 37))) + [span - 1, span, span + 1, 10 ** 9]:
            assert B.d3_depth_linear(upper, lower, span, i) == O.depth_linear(upper, lower, span, i)
    for bad in [(-1, 0, 5, 0), (4, 5, 5, 0), (4, -1, 5, 0), (4, 0, 0, 0), (4, 0, 5, -1)]:
        assert B.d3_depth_linear(*bad) == B.EINVAL
    assert B.LIB.d3_decode_step_depths(None, 1, None, None, None, None, None, None) == B.EINVAL
