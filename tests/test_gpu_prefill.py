"""Batched full-depth prefill (initiation phase, Sec. 3.1; Sec. 4.1 "passing prompt inputs
through all layers"): passes of up to 128 prompt positions through tensor-core projections and
the causal flash-attention kernel, against the CPU oracle (GPU)."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2503_08524_b200 import inputs as I

from parity import LOGITS_MAX_ABS, check_step, make_pair, rel_l2

pytestmark = pytest.mark.gpu
SEED = I.BASE_SEED + 60


def _compare_cache(orc, gpu, shape, slot, positions, tol=2e-2):
    for l in range(shape.n_layers):
        for t in positions:
            ok, ov = orc.read_kv(l, slot, t)
            gk, gv = gpu.d3_read_kv(l, slot, t)
            assert np.abs(gk - ok).max() < tol and np.abs(gv - ov).max() < tol, (l, t)


@pytest.mark.parametrize("shape", [I.TINY, I.TINY_GQA], ids=["mha-64", "gqa-32"])
@pytest.mark.parametrize("paged", [False, True], ids=["contiguous", "paged"])
@pytest.mark.parametrize("exec_mode", [0, 1], ids=["auto", "kernels"])
def test_prefill_passes_of_128_positions(shape, paged, exec_mode):
    """Ragged prompt lengths around the pass and tile boundaries: logits, final hidden state and
    the cache contents of every block; then decode steps that read the prefilled cache."""
    pk = dict(page_size=32, n_pages=1 + shape.n_layers * 24) if paged else {}
    orc, gpu = make_pair(shape, SEED, 2, 448, 128, start_id=1, **pk)
    gpu.d3_set_exec(exec_mode)
    for slot, n in [(0, 7), (1, 8), (0, 128), (1, 129), (0, 145), (1, 300), (0, 401)]:
        p = I.prompt_tokens(shape, SEED, slot * 1000 + n, n).numpy()
        o, oh = orc.prefill(slot, p, want_hidden=True)
        g = gpu.d3_prefill(slot, p)
        check_step(f"prefill {n}", g.cpu().numpy()[None], None, o[None], None)
        assert gpu.d3_slot_pos(slot) == n
        _compare_cache(orc, gpu, shape, slot, sorted({0, n // 3, n // 2, max(0, n - 17), n - 1}))
    # both slots go on decoding over what the prefill cached
    for i in range(1, 4):
        toks = I.token_ids(SEED, 70 + i, 2, shape.vocab).numpy()
        r = orc.decode_step([0, 1], toks, [i, i + 9], 0.93)
        g = gpu.d3_decode_step([0, 1], toks, [i, i + 9], 0.93)
        check_step(f"step {i}", g.cpu().numpy(), gpu.d3_read_hidden(2), r["logits"], r["hidden"])
    gpu.d3_sync()
    gpu.close()


@pytest.mark.parametrize("base,layers,n", [(I.LLAMA_7B, 2, 200), (I.LLAMA_70B, 2, 150), (I.LLAMA_13B, 1, 131)],
                         ids=["7b-width", "70b-width-gqa", "13b-width"])
def test_prefill_at_production_widths(base, layers, n):
    """Full-width blocks (two operand groups of 64 positions, head_dim 128, 1 and 8 query heads per
    KV head): prefill logits and the hidden state of the last position, then two decode steps."""
    shape = base.with_layers(layers)
    orc, gpu = make_pair(shape, SEED + 1, 1, n + 8, 128, start_id=0)
    p = I.prompt_tokens(shape, SEED + 1, 0, n).numpy()
    o, oh = orc.prefill(0, p, want_hidden=True)
    g = gpu.d3_prefill(0, p)
    check_step("prefill", g.cpu().numpy()[None], None, o[None], None)
    assert rel_l2(gpu.d3_read_hidden(128)[(n - 1) % 128], oh) <= 1e-2
    _compare_cache(orc, gpu, shape, 0, [0, 63, 64, 127, 128, n - 1], tol=4e-2)
    for i in (1, 2):
        r = orc.decode_step([0], [5 + i], [i], 1.0)
        g = gpu.d3_decode_step([0], [5 + i], [i], 1.0)
        check_step(f"step {i}", g.cpu().numpy(), gpu.d3_read_hidden(1), r["logits"], r["hidden"])
    gpu.d3_sync()
    gpu.close()


def test_hundred_twenty_eight_rows_per_decode_step():
    """The widest step the ABI allows: 128 rows of mixed depths (two operand groups in every
    projection), and one row too many is refused."""
    from paper_2503_08524_b200 import binding as B
    shape = I.TINY_GQA
    Bn, L = 128, shape.n_layers
    orc, gpu = make_pair(shape, SEED + 2, Bn, 64, Bn, start_id=0, kv_fill=1)
    for b in range(Bn):
        n = 1 + (11 * b) % 40
        p = I.prompt_tokens(shape, SEED + 2, b, n).numpy()
        orc.prefill(b, p)
        gpu.d3_prefill(b, p)
    for step in range(2):
        toks = I.token_ids(SEED + 2, 70 + step, Bn, shape.vocab).numpy()
        gi = [1 + step + (b % 70) for b in range(Bn)]
        r = orc.decode_step(list(range(Bn)), toks, gi, 0.955)
        g, st = gpu.d3_decode_step(list(range(Bn)), toks, gi, 0.955, want_stats=True)
        check_step(f"step {step}", g.cpu().numpy(), gpu.d3_read_hidden(Bn), r["logits"], r["hidden"])
        want = O.schedule(L, 0.955, 0, 0, gi)
        assert np.array_equal(st["n"], want["n"]) and np.array_equal(st["m_per_layer"], want["m_per_layer"])
    with pytest.raises(B.D3Error) as e:
        gpu.d3_decode_step(list(range(Bn)) + [0], [1] * 129, [1] * 129, 1.0)
    assert e.value.code == B.ECAPACITY
    gpu.d3_sync()
    gpu.close()
