"""The oracle's window policy changed between steps (`start`, anchor and fill differ per task:
Sec. 4.1, "Hyperparameter Settings"), pinned on the CPU: a switched oracle must behave exactly like
one built with the new policy, and like a hand-listed stack of the blocks outside the new window."""
import numpy as np
import pytest

import oracle as O
from paper_2503_08524_b200 import inputs as I

SEED = I.BASE_SEED + 70


def _pair(policy_a, policy_b, max_seq=48):
    shape = I.TINY
    w = I.make_weights(shape, SEED, device="cpu", gain_jitter=0.1)
    a = O.Oracle(shape, w, 1, max_seq, start_id=policy_a[0], anchor=policy_a[1], kv_fill=policy_a[2])
    b = O.Oracle(shape, w, 1, max_seq, start_id=policy_b[0], anchor=policy_b[1], kv_fill=policy_b[2])
    prompt = I.prompt_tokens(shape, SEED, 0, 9).numpy()
    la, lb = a.prefill(0, prompt), b.prefill(0, prompt)
    assert (la == lb).all()                      # the prompt runs all blocks whatever the policy
    tok = O.argmax(la)
    for i in (1, 2):                             # full-depth steps: empty windows, policy-free caches
        ra = a.decode_step([0], [tok], [i], 1.0)
        rb = b.decode_step([0], [tok], [i], 1.0)
        assert (ra["logits"] == rb["logits"]).all()
        tok = O.argmax(ra["logits"][0])
    return shape, a, b, tok


@pytest.mark.parametrize("new", [(2, O.ANCHOR_START, O.FILL_COPY), (0, O.ANCHOR_TAIL, O.FILL_RECOMPUTE),
                                 (1, O.ANCHOR_START, O.FILL_NONE), (3, O.ANCHOR_START, O.FILL_COPY)])
def test_switched_oracle_equals_one_built_with_the_new_policy(new):
    shape, a, b, tok = _pair((0, O.ANCHOR_START, O.FILL_COPY), new)
    a.set_policy(*new)
    for i in (3, 9, 20):                         # depths 3, 2, 1 of 4 at alpha 0.93
        ra = a.decode_step([0], [tok], [i], 0.93)
        rb = b.decode_step([0], [tok], [i], 0.93)
        assert (ra["logits"] == rb["logits"]).all() and (ra["hidden"] == rb["hidden"]).all()
        for l in range(shape.n_layers):
            ka, va = a.read_kv(l, 0, a.slot_pos(0) - 1)
            kb, vb = b.read_kv(l, 0, b.slot_pos(0) - 1)
            assert np.array_equal(ka, kb, equal_nan=True) and np.array_equal(va, vb, equal_nan=True)
        tok = O.argmax(ra["logits"][0])


@pytest.mark.parametrize("start,anchor", [(2, O.ANCHOR_START), (1, O.ANCHOR_START), (0, O.ANCHOR_TAIL)])
def test_step_after_a_switch_runs_the_blocks_outside_the_new_window(start, anchor):
    # the twin takes the same step as a hand-listed stack (no schedule code involved)
    shape, a, twin, tok = _pair((0, O.ANCHOR_START, O.FILL_NONE), (0, O.ANCHOR_START, O.FILL_NONE))
    L = shape.n_layers
    a.set_policy(start, anchor, O.FILL_NONE)
    i, alpha = 9, 0.93
    n, lo, hi = O.window(L, alpha, i, start, anchor)
    assert 0 < hi - lo < L                       # a real window
    r = a.decode_step([0], [tok], [i], alpha)
    logits, hidden = twin.decode_layers(0, tok, [l for l in range(L) if not (lo <= l < hi)])
    assert (r["logits"][0] == logits).all() and (r["hidden"][0] == hidden).all()
