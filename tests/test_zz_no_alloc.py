"""The allocation-free decode step (d3_decode_step_noalloc) against the CPU oracle and the regular step.

Some callers of this library may not allocate device memory when they decode:
a plugin inside an application that owns the GPU's memory, a loop that must not
allocate after start-up, a process at its memory limit.  For them the library
carries its scratch in a fixed array of its own.  This file checks, through the
C ABI, that the step on that array gives what the oracle computes and leaves
the cache that d3_decode_step leaves on caller-provided scratch, twice in a row (the array keeps the first call's
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


@pytest.mark.parametrize("shape,max_seq,plen,start", [(I.TINY, 96, 37, 1), (I.LLAMA_7B.with_layers(3), 128, 21, 1)],
                         ids=["tiny", "7b-width-3-blocks"])
def test_noalloc_step_equals_oracle_and_regular_step_twice_in_a_row(shape, max_seq, plen, start):
    """Two steps in a row on the built-in array (the second finds the first one's contents
    there), each checked against the CPU oracle at the tolerances of every other parity test,
    and against the regular entry point's cache.  The 7B-width case puts the attention
    partials and the activations megabytes into the array, not kilobytes."""
    from paper_2503_08524_b200 import binding as B
    import oracle as O
    dev = "cuda:0"
    seed = I.BASE_SEED + 11
    w = I.make_weights(shape, seed, device=dev, gain_jitter=0.1)
    orc = O.Oracle(shape, I.weights_to(w, "cpu"), 2, max_seq, start_id=start, kv_fill=B.FILL_COPY,
                   kv_round_bf16=True)
    ref = B.D3Model(shape, w, 2, max_seq, 1, start_id=start, kv_fill=B.FILL_COPY, device=dev)
    ref.zero_kv()
    cfg = B.make_config(shape, 2, max_seq, 1, start_id=start, kv_fill=B.FILL_COPY)
    assert B.d3_workspace_bytes(cfg)[1] <= B.NOALLOC_SCRATCH_BYTES
    # a second KV cache for the allocation-free path, filled by the same prefill
    prompt = I.prompt_tokens(shape, seed, 0, plen).numpy()
    orc.prefill(1, prompt)
    ref.d3_prefill(1, prompt)
    ref.d3_sync()
    kv2 = ref.kv.clone()
    logits2 = torch.empty(shape.vocab, dtype=torch.float32, device=dev)
    toks = I.token_ids(seed, 3, 4, shape.vocab).numpy()
    pos = len(prompt)
    L = shape.n_layers
    steps = [(1, 0.9), (7, 0.9)] if L == 4 else [(1, 0.8), (3, 0.8)]    # depths 3, 1 of 4 / 2, 1 of 3
    for call, (i, alpha) in enumerate(steps):
        want = orc.decode_step([1], [int(toks[call])], [i], alpha)["logits"][0]
        ref.d3_decode_step([1], [int(toks[call])], [i], alpha)
        rc = B.d3_decode_step_noalloc(cfg, w, kv2, 1, pos, int(toks[call]), i, alpha, logits2)
        assert rc == B.OK, B.strerror(rc)
        assert B.d3_noalloc_status() == B.OK          # waits for the stream; no device-side time-out
        got = logits2.cpu().numpy()
        assert np.isfinite(got).all()
        assert np.abs(got - want).max() <= LOGITS_MAX_ABS, (call, np.abs(got - want).max())
        # both entry points left the same cache behind (retained blocks and the copy fill)
        ref.d3_sync()
        assert torch.equal(kv2, ref.kv), call
        pos += 1
    ref.close()
    orc.close()


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
