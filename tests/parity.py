"""Shared machinery of the GPU parity tests: the same seeded inputs go to the
CPU oracle and, through the C ABI, to the CUDA library; outputs are compared
element by element."""
import numpy as np
import torch

import oracle as O
from paper_2503_08524_b200 import inputs as I

# Tolerances of the float comparisons (bf16 weights and KV cache, fp32
# activations and accumulation on the GPU; fp64 oracle on the same bf16 weights).
LOGITS_MAX_ABS = 2e-2
HIDDEN_REL_L2 = 1e-2


def rel_l2(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30))


def make_pair(shape, seed, max_slots, max_seq, max_batch, start_id=0, anchor=0, kv_fill=1,
              gain_jitter=0.1, gen_device="cuda:0", kv_round_bf16=True, page_size=0, n_pages=0):
    """(oracle, gpu model) over identical weights.  Weights are generated once
    (integer hash, bit-identical on either device) and copied to the other side.
    kv_round_bf16: the oracle stores K and V rounded to bf16, the cache format
    of the GPU path (the storage precision is part of the data layout; at 4096+
    widths the rounding alone moves logits by more than the tolerance, so both
    sides must store alike).  The tiny-config run also passes without it."""
    from paper_2503_08524_b200 import binding as B
    w_dev = I.make_weights(shape, seed, device=gen_device, gain_jitter=gain_jitter)
    w_cpu = I.weights_to(w_dev, "cpu")
    orc = O.Oracle(shape, w_cpu, max_slots, max_seq, start_id=start_id, anchor=anchor, kv_fill=kv_fill,
                   kv_round_bf16=kv_round_bf16)
    gpu = B.D3Model(shape, w_dev, max_slots, max_seq, max_batch, start_id=start_id, anchor=anchor,
                    kv_fill=kv_fill, page_size=page_size, n_pages=n_pages)
    return orc, gpu


def check_step(tag, g_logits, g_hidden, o_logits, o_hidden):
    g_logits = np.asarray(g_logits, np.float64)
    assert np.isfinite(g_logits).all(), tag
    err = np.abs(g_logits - o_logits).max()
    assert err <= LOGITS_MAX_ABS, (tag, "logits max-abs", err)
    if g_hidden is not None:
        for b in range(o_hidden.shape[0]):
            r = rel_l2(g_hidden[b], o_hidden[b])
            assert r <= HIDDEN_REL_L2, (tag, "hidden rel-L2", b, r)
    return err
