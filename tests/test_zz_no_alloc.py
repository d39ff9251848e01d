"""The allocation-free decode step (d3_decode_step_noalloc) against the regular one.

Some callers of this library may not allocate device memory when they decode:
a plugin inside an application that owns the GPU's memory, a loop that must not
allocate after start-up, a process at its memory limit.  For them the library
carries its scratch in a fixed array of its own.  This file checks, through the
C ABI, that the step on that array gives what d3_decode_step gives on
caller-provided scratch, twice in a row (the array keeps the first call's
contents when the second one starts), and that oversized or unsupported
requests are refused with an error code instead of being attempted.

The file sorts last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2503_08524_b200 import inputs as I

from parity import LOGITS_MAX_ABS

pytestmark = pytest.mark.gpu


def test_noalloc_step_equals_regular_step_twice_in_a_row():
    from paper_2503_08524_b200 import binding as B
    shape = I.TINY
    dev = "cuda:0"
    w = I.make_weights(shape, I.BASE_SEED + 11, device=dev, gain_jitter=0.1)
    max_seq = 96
    ref = B.D3Model(shape, w, 2, max_seq, 1, start_id=1, kv_fill=B.FILL_COPY, device=dev)
    ref.zero_kv()
    cfg = B.make_config(shape, 2, max_seq, 1, start_id=1, kv_fill=B.FILL_COPY)
    # a second KV cache for the allocation-free path, filled by the same prefill
    prompt = I.prompt_tokens(shape, I.BASE_SEED + 11, 0, 37).numpy()
    ref.d3_prefill(1, prompt)
    ref.d3_sync()
    kv2 = ref.kv.clone()
    logits2 = torch.empty(shape.vocab, dtype=torch.float32, device=dev)
    toks = I.token_ids(I.BASE_SEED + 11, 3, 4, shape.vocab).numpy()
    pos = len(prompt)
    for call, (i, alpha) in enumerate([(1, 0.9), (7, 0.9)]):      # depths 3 and 1 of 4
        want = ref.d3_decode_step([1], [int(toks[call])], [i], alpha).cpu().numpy()[0]
        rc = B.d3_decode_step_noalloc(cfg, w, kv2, 1, pos, int(toks[call]), i, alpha, logits2)
        assert rc == B.OK, B.strerror(rc)
        torch.cuda.synchronize()
        got = logits2.cpu().numpy()
        assert np.isfinite(got).all()
        assert np.abs(got - want).max() <= LOGITS_MAX_ABS, (call, np.abs(got - want).max())
        # both paths left the same cache behind (retained blocks and the copy fill)
        assert torch.equal(kv2, ref.kv), call
        pos += 1
    ref.close()


def test_noalloc_step_refuses_what_it_cannot_serve():
    from paper_2503_08524_b200 import binding as B
    shape = I.TINY
    dev = "cuda:0"
    w = I.make_weights(shape, I.BASE_SEED + 12, device=dev)
    cfg = B.make_config(shape, 1, 64, 1)
    kv_bytes, _ = B.d3_workspace_bytes(cfg)
    kv = torch.zeros(kv_bytes, dtype=torch.uint8, device=dev)
    lg = torch.empty(shape.vocab, dtype=torch.float32, device=dev)
    ok = dict(slot=0, pos=5, token=3, gen_index=1, alpha=0.9)

    def call(c=cfg, **kw):
        a = dict(ok)
        a.update(kw)
        return B.d3_decode_step_noalloc(c, w, kv, a["slot"], a["pos"], a["token"], a["gen_index"],
                                        a["alpha"], lg)

    assert call(pos=0) == B.EINVAL and call(gen_index=0) == B.EINVAL
    assert call(token=shape.vocab) == B.EINVAL and call(slot=1) == B.EINVAL
    assert call(alpha=0.0) == B.EINVAL and call(alpha=float("nan")) == B.EINVAL
    assert call(pos=64) == B.ECAPACITY
    # a cache so long that one row's scratch (rotary table) exceeds the fixed array
    big = B.make_config(shape, 1, 1 << 16, 1)
    assert B.d3_workspace_bytes(big)[1] > B.NOALLOC_SCRATCH_BYTES
    assert call(c=big) == B.ECAPACITY
    recompute = B.make_config(shape, 1, 64, 1, kv_fill=B.FILL_RECOMPUTE)
    assert call(c=recompute) == B.EINVAL
    assert call() == B.OK
    torch.cuda.synchronize()
