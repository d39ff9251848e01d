"""Window policy changed between steps, and the bounded-wait time-out path (GPU)."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2503_08524_b200 import inputs as I

from parity import check_step, make_pair

pytestmark = pytest.mark.gpu
SEED = I.BASE_SEED + 40


@pytest.mark.parametrize("exec_mode", [0, 1], ids=["auto", "kernels"])
def test_policy_changed_between_steps(exec_mode):
    """`start`, anchor and fill differ per task (Sec. 4.1, "Hyperparameter Settings"): the same
    sequences go on under a new policy from the next step, on both sides."""
    from paper_2503_08524_b200 import binding as B
    shape = I.TINY
    orc, gpu = make_pair(shape, SEED, 3, 96, 3, start_id=0, anchor=0, kv_fill=1)
    gpu.d3_set_exec(exec_mode)
    orc.poison_kv()
    gpu.poison_kv()             # an entry nobody wrote is NaN on both sides
    for s in range(3):
        p = I.prompt_tokens(shape, SEED, s, 6 + 7 * s).numpy()
        orc.prefill(s, p)
        gpu.d3_prefill(s, p)
    policies = [(0, 0, 1), (2, 0, 1), (1, 0, 2), (0, 1, 1), (3, 0, 1), (1, 0, 0)]   # fill NONE last
    step = 0
    for start, anchor, fill in policies:
        orc.set_policy(start, anchor, fill)
        gpu.d3_set_policy(start, anchor, fill)
        for rows in ([0, 1, 2], [1]):          # a mixed-depth batch, then one row alone
            toks = I.token_ids(SEED, 100 + step, len(rows), shape.vocab).numpy()
            gi = [2 + 5 * step + 9 * b for b in range(len(rows))]
            r = orc.decode_step(rows, toks, gi, 0.93)
            g, st = gpu.d3_decode_step(rows, toks, gi, 0.93, want_stats=True)
            want = O.schedule(shape.n_layers, 0.93, start, anchor, gi)
            assert np.array_equal(st["n"], want["n"])
            assert np.array_equal(st["m_per_layer"], want["m_per_layer"])
            check_step((start, anchor, fill, rows), g.cpu().numpy(), gpu.d3_read_hidden(len(rows)),
                       r["logits"], r["hidden"])
            step += 1
    # the caches agree entry by entry wherever the oracle's entry is defined
    for s in range(3):
        for l in range(shape.n_layers):
            for t in range(orc.slot_pos(s)):
                ok, ov = orc.read_kv(l, s, t)
                gk, gv = gpu.d3_read_kv(l, s, t)
                m = np.isfinite(ok)
                assert np.abs(gk[m] - ok[m]).max(initial=0) < 2e-2 and np.abs(gv[m] - ov[m]).max(initial=0) < 2e-2
    with pytest.raises(B.D3Error):
        gpu.d3_set_policy(shape.n_layers + 1, 0, 1)
    with pytest.raises(B.D3Error):
        gpu.d3_set_policy(0, 2, 1)
    with pytest.raises(B.D3Error):
        gpu.d3_set_policy(0, 0, 3)
    gpu.d3_sync()
    gpu.close()


def test_wait_that_nobody_satisfies_times_out_and_the_model_recovers():
    """Failure detection without a fault: the host tells one single-kernel step to expect an
    arrival at its first grid barrier that never comes and gives the waits a 3 ms limit.  The
    kernel must give up, report D3_ETIMEOUT through d3_sync, and leave the GPU and the model
    usable: after a reset and a new prefill the next steps match the oracle again."""
    from paper_2503_08524_b200 import binding as B
    shape = I.TINY
    orc, gpu = make_pair(shape, SEED + 1, 1, 64, 1, start_id=1)
    prompt = I.prompt_tokens(shape, SEED + 1, 0, 11).numpy()
    gpu.d3_prefill(0, prompt)
    gpu.d3_set_exec(B.EXEC_FUSED)
    # a healthy step first
    orc.prefill(0, prompt)
    r = orc.decode_step([0], [5], [1], 0.9)
    g = gpu.d3_decode_step([0], [5], [1], 0.9)
    check_step("before", g.cpu().numpy(), gpu.d3_read_hidden(1), r["logits"], r["hidden"])
    gpu.d3_sync()
    # the drill
    gpu.d3_set_wait_ns(3_000_000)
    gpu.d3_stall_next_step()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    _, st = gpu.d3_decode_step([0], [7], [2], 0.9, want_stats=True)
    ev1.record()
    assert st["kernel_launches"] == 1
    with pytest.raises(B.D3Error) as e:
        gpu.d3_sync()
    assert e.value.code == B.ETIMEOUT
    ms = ev0.elapsed_time(ev1)
    assert 2.5 < ms < 500.0, ms          # it waited its limit, not forever
    gpu.d3_sync()                        # reported once, then clear
    # recovery: default limit, fresh slot, same sequence as the oracle's
    gpu.d3_set_wait_ns(2_000_000_000)
    gpu.d3_reset_slot(0)
    gpu.d3_prefill(0, prompt)
    g = gpu.d3_decode_step([0], [5], [1], 0.9)          # the oracle already took this step
    assert np.abs(g.cpu().numpy() - r["logits"]).max() <= 2e-2
    for i, tok in ((2, 7), (3, 9)):
        r = orc.decode_step([0], [tok], [i], 0.9)
        g = gpu.d3_decode_step([0], [tok], [i], 0.9)
        check_step(("after", i), g.cpu().numpy(), gpu.d3_read_hidden(1), r["logits"], r["hidden"])
    gpu.d3_sync()
    with pytest.raises(B.D3Error):
        gpu.d3_set_wait_ns(0)
    gpu.close()
