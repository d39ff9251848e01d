"""Pins of the oracle's decoder, cache and skipped-layer handling (no GPU)."""
import math

import numpy as np
import pytest
import torch

import oracle as O
from paper_2503_08524_b200 import inputs as I

from hf_llama import build as hf_build, only_layers

SEED = I.BASE_SEED
HF_TOL = 2e-6      # the library builds its rotary tables in fp32


def make(shape, **kw):
    w = I.make_weights(shape, SEED, gain_jitter=0.1)
    return w, O.Oracle(shape, w, kw.pop("max_slots", 4), kw.pop("max_seq", 96), **kw)


@pytest.fixture(scope="module", params=[I.TINY, I.TINY_GQA], ids=["mha", "gqa"])
def setup(request):
    shape = request.param
    w = I.make_weights(shape, SEED, gain_jitter=0.1)
    hf, cfg = hf_build(shape, w)
    toks = I.prompt_tokens(shape, SEED, 0, 40)
    with torch.no_grad():
        out = hf(input_ids=toks.long()[None], output_hidden_states=True)
    return shape, w, hf, cfg, toks, out


def test_full_depth_equals_library_llama(setup):
    shape, w, hf, cfg, toks, out = setup
    ref = out.logits[0].numpy()
    orc = O.Oracle(shape, w, 2, 64, start_id=1)
    lg = orc.prefill(1, toks[:16].numpy())
    assert np.abs(lg - ref[15]).max() < HF_TOL
    for p in range(16, 40):                       # alpha = 1: every step is the full model
        r = orc.decode_step([1], [int(toks[p])], [p - 15], 1.0)
        assert np.abs(r["logits"][0] - ref[p]).max() < HF_TOL
    assert orc.slot_pos(1) == 40


def test_cached_decode_equals_forward_without_cache(setup):
    shape, w, hf, cfg, toks, out = setup
    orc = O.Oracle(shape, w, 1, 64)
    nc = orc.forward_nocache(toks[:24].numpy())
    assert np.abs(nc - out.logits[0, :24].numpy()).max() < HF_TOL
    lg = orc.prefill(0, toks[:10].numpy())
    assert np.abs(lg - nc[9]).max() < 1e-11
    for p in range(10, 24):
        r = orc.decode_step([0], [int(toks[p])], [p - 9], 1.0)
        assert np.abs(r["logits"][0] - nc[p]).max() < 1e-11


def test_tail_truncation_equals_library_hidden_state(setup):
    # Early-Exit direction: a token that keeps its first n blocks yields
    # lm_head(norm(h^n)), h^n the library's hidden state after block n.
    shape, w, hf, cfg, toks, out = setup
    L = shape.n_layers
    for n_keep, alpha in [(4, 1.0), (3, 0.8), (2, 0.7), (1, 0.4), (0, 0.2)]:
        assert O.depth(L, alpha, 1) == n_keep
        orc = O.Oracle(shape, w, 1, 64, anchor=O.ANCHOR_TAIL, kv_fill=O.FILL_NONE)
        orc.prefill(0, toks[:20].numpy())
        r = orc.decode_step([0], [int(toks[20])], [1], alpha, want_trace=True)
        h_n = out.hidden_states[n_keep][0, 20] if n_keep < L else None
        if n_keep < L:
            # hidden_states[k] for k < L is the raw residual stream after k blocks
            assert np.abs(r["hidden"][0] - h_n.numpy()).max() < HF_TOL
            with torch.no_grad():
                want = hf.lm_head(hf.model.norm(h_n)).numpy()
        else:
            want = out.logits[0, 20].numpy()
        assert np.abs(r["logits"][0] - want).max() < HF_TOL
        for k in range(n_keep + 1):
            if k < L:
                assert np.abs(r["trace"][0, k] - out.hidden_states[k][0, 20].numpy()).max() < HF_TOL


def test_saturation_probe_equals_library_per_block_predictions(setup):
    # Sec. 3.2: for the token at one position, what lm_head predicts from every block's output.
    # The library gives the same from its hidden states: argmax and softmax of
    # lm_head(norm(hidden_states[i])) for i < L, of its final logits for i = L.
    shape, w, hf, cfg, toks, out = setup
    L = shape.n_layers
    orc = O.Oracle(shape, w, 1, 64)
    orc.prefill(0, toks[:20].numpy())
    r = orc.saturation_probe([0], [int(toks[20])])
    assert orc.slot_pos(0) == 21 and r["tokens"].shape == (1, L)
    for i in range(1, L + 1):
        with torch.no_grad():
            lg = (hf.lm_head(hf.model.norm(out.hidden_states[i][0, 20])) if i < L else out.logits[0, 20]).double()
        p = torch.softmax(lg, -1)
        assert r["tokens"][0, i - 1] == int(torch.argmax(lg))
        assert abs(r["conf"][0, i - 1] - float(p.max())) < 1e-6
    assert r["tokens"][0, L - 1] == O.argmax(r["logits"][0])
    # closed form: a state whose logits are all equal has confidence 1 / vocab, token 0
    tok, conf, lg = orc.probe(np.zeros(shape.d_model))
    assert tok == 0 and abs(conf - 1.0 / shape.vocab) < 1e-12 and np.all(lg == 0.0)


@pytest.mark.parametrize("anchor,start,alpha", [(O.ANCHOR_START, 1, 0.93), (O.ANCHOR_START, 2, 0.9),
                                                (O.ANCHOR_TAIL, 0, 0.95), (O.ANCHOR_START, 3, 0.8)])
@pytest.mark.parametrize("fill", [O.FILL_NONE, O.FILL_COPY, O.FILL_RECOMPUTE])
def test_depth_decay_run_equals_library_with_layers_deleted(setup, anchor, start, alpha, fill):
    # The paper's own construction: the library model, per generated token, with
    # the dropped layers removed and the KV cache kept.  Teacher-forced tokens.
    from transformers.cache_utils import DynamicCache
    shape, w, hf, cfg, toks, out = setup
    L, P = shape.n_layers, 12
    orc = O.Oracle(shape, w, 1, 64, start_id=start, anchor=anchor, kv_fill=fill)
    orc.poison_kv()
    lg0 = orc.prefill(0, toks[:P].numpy())
    cache = DynamicCache(config=cfg)
    with torch.no_grad():
        o = hf(input_ids=toks[:P].long()[None], past_key_values=cache, use_cache=True)
    assert np.abs(lg0 - o.logits[0, -1].numpy()).max() < HF_TOL
    depths = []
    for i in range(1, 25):
        n, lo, hi = O.window(L, alpha, i, start, anchor)
        keep = [l for l in range(L) if not (lo <= l < hi)]
        if not keep or keep[0] != 0:
            break                                   # the library sizes its mask from layer 0
        depths.append(n)
        tok = int(toks[P + i - 1])
        with only_layers(hf, keep), torch.no_grad():
            o = hf(input_ids=torch.tensor([[tok]]), past_key_values=cache, use_cache=True)
        r = orc.decode_step([0], [tok], [i], alpha)
        assert np.abs(r["logits"][0] - o.logits[0, 0].numpy()).max() < HF_TOL, (i, keep)
    assert len(depths) >= 8 and depths[-1] < L          # the run did shed layers


def test_alpha_one_is_the_plain_full_decode():
    for shape in (I.TINY, I.TINY_GQA):
        w = I.make_weights(shape, SEED + 1, gain_jitter=0.1)
        toks = I.prompt_tokens(shape, SEED + 1, 0, 30)
        ref = O.Oracle(shape, w, 1, 48)
        ref.prefill(0, toks[:8].numpy())
        variants = [O.Oracle(shape, w, 1, 48, start_id=s, anchor=a, kv_fill=f)
                    for s, a, f in [(0, 0, 0), (2, 0, 1), (4, 0, 2), (1, 1, 1), (3, 1, 2)]]
        for v in variants:
            v.prefill(0, toks[:8].numpy())
        for p in range(8, 30):
            lg, hid = ref.decode_layers(0, int(toks[p]), list(range(shape.n_layers)))
            for v in variants:
                r = v.decode_step([0], [int(toks[p])], [p - 7], 1.0)
                assert np.array_equal(r["logits"][0], lg) and np.array_equal(r["hidden"][0], hid)


@pytest.mark.parametrize("anchor,start", [(O.ANCHOR_START, 0), (O.ANCHOR_START, 1), (O.ANCHOR_START, 3),
                                          (O.ANCHOR_TAIL, 0)])
def test_scheduled_step_equals_hand_truncated_stack(anchor, start):
    shape = I.TINY_GQA
    w = I.make_weights(shape, SEED + 2, gain_jitter=0.1)
    toks = I.prompt_tokens(shape, SEED + 2, 0, 40)
    L, alpha = shape.n_layers, 0.9
    a = O.Oracle(shape, w, 1, 64, start_id=start, anchor=anchor, kv_fill=O.FILL_NONE)
    b = O.Oracle(shape, w, 1, 64)
    a.prefill(0, toks[:6].numpy())
    b.prefill(0, toks[:6].numpy())
    seen = set()
    for i in range(1, 30):
        n, lo, hi = O.window(L, alpha, i, start, anchor)
        keep = [l for l in range(L) if not (lo <= l < hi)]
        seen.add(n)
        tok = int(toks[5 + i])
        r = a.decode_step([0], [tok], [i], alpha)
        lg, hid = b.decode_layers(0, tok, keep)
        assert np.array_equal(r["logits"][0], lg) and np.array_equal(r["hidden"][0], hid)
    assert len(seen) >= (3 if start < 2 else 1)
    if start == 0 or anchor == O.ANCHOR_TAIL:
        assert 0 in seen          # depth 0: logits of the bare embedding


@pytest.mark.parametrize("anchor,start,fill", [(O.ANCHOR_START, 1, O.FILL_COPY), (O.ANCHOR_START, 0, O.FILL_NONE),
                                               (O.ANCHOR_TAIL, 0, O.FILL_RECOMPUTE)])
def test_step_with_given_depths_equals_the_alpha_step_and_the_truncated_stack(anchor, start, fill):
    # (a) depths = floor(L alpha^i) must reproduce the alpha step bit for bit (logits, hidden,
    #     cache); (b) any other depth sequence (here: linear decay) must equal the stack with
    #     the window's blocks removed by hand.
    shape = I.TINY_GQA
    w = I.make_weights(shape, SEED + 6, gain_jitter=0.1)
    toks = I.prompt_tokens(shape, SEED + 6, 0, 48).numpy()
    L, alpha = shape.n_layers, 0.92
    a = O.Oracle(shape, w, 2, 64, start_id=start, anchor=anchor, kv_fill=fill)
    b = O.Oracle(shape, w, 2, 64, start_id=start, anchor=anchor, kv_fill=fill)
    for orc in (a, b):
        orc.prefill(0, toks[:5])
        orc.prefill(1, toks[:9])
    for i in range(1, 20):
        gi = [i, i + 4]
        tk = [int(toks[10 + i]), int(toks[20 + i])]
        ra = a.decode_step([0, 1], tk, gi, alpha)
        rb = b.decode_step_depths([0, 1], tk, [O.depth(L, alpha, g) for g in gi])
        assert np.array_equal(ra["logits"], rb["logits"]) and np.array_equal(ra["hidden"], rb["hidden"])
    for l in range(L):
        for slot in (0, 1):
            ka, va = a.read_kv(l, slot, a.slot_pos(slot) - 1)
            kb, vb = b.read_kv(l, slot, b.slot_pos(slot) - 1)
            assert np.array_equal(ka, kb, equal_nan=True) and np.array_equal(va, vb, equal_nan=True)
    # (b) linear decay, one row, against the hand-truncated stack (nothing filled on that side)
    c = O.Oracle(shape, w, 1, 64, start_id=start, anchor=anchor, kv_fill=O.FILL_NONE)
    d = O.Oracle(shape, w, 1, 64)
    c.prefill(0, toks[:6])
    d.prefill(0, toks[:6])
    seen = set()
    for i in range(1, 16):
        n = O.depth_linear(L, 1, 12, i)
        nn, lo, hi = O.window_of_depth(L, n, start, anchor)
        seen.add(nn)
        keep = [l for l in range(L) if not (lo <= l < hi)]
        tok = int(toks[6 + i])
        r = c.decode_step_depths([0], [tok], [n])
        lg, hid = d.decode_layers(0, tok, keep)
        assert np.array_equal(r["logits"][0], lg) and np.array_equal(r["hidden"][0], hid)
    assert len(seen) >= 3
    with pytest.raises(ValueError):
        c.decode_step_depths([0], [1], [L + 1])


@pytest.mark.parametrize("anchor", [O.ANCHOR_START, O.ANCHOR_TAIL])
def test_logits_do_not_depend_on_the_fill_mode(anchor):
    # depth never grows along a sequence, so no later token reads an entry that
    # a skipped layer left (NaN-poisoned under FILL_NONE)
    shape = I.TINY
    w = I.make_weights(shape, SEED + 3, gain_jitter=0.1)
    toks = I.prompt_tokens(shape, SEED + 3, 0, 50)
    runs = []
    for fill in (O.FILL_NONE, O.FILL_COPY, O.FILL_RECOMPUTE):
        orc = O.Oracle(shape, w, 1, 64, start_id=1 if anchor == O.ANCHOR_START else 0,
                       anchor=anchor, kv_fill=fill)
        orc.poison_kv()
        out = [orc.prefill(0, toks[:10].numpy())]
        for i in range(1, 40):
            out.append(orc.decode_step([0], [int(toks[9 + i])], [i], 0.95)["logits"][0])
        runs.append(np.stack(out))
        assert np.isfinite(runs[-1]).all()
    assert np.array_equal(runs[0], runs[1]) and np.array_equal(runs[0], runs[2])


def test_fill_modes_write_what_they_say():
    shape = I.TINY_GQA
    w = I.make_weights(shape, SEED + 4, gain_jitter=0.1)
    toks = I.prompt_tokens(shape, SEED + 4, 0, 20)
    L = shape.n_layers
    for start, anchor in [(2, O.ANCHOR_START), (0, O.ANCHOR_START), (0, O.ANCHOR_TAIL)]:
        cache = {}
        for fill in (O.FILL_NONE, O.FILL_COPY, O.FILL_RECOMPUTE):
            orc = O.Oracle(shape, w, 1, 32, start_id=start, anchor=anchor, kv_fill=fill)
            orc.poison_kv()
            orc.prefill(0, toks[:8].numpy())
            r = orc.decode_step([0], [int(toks[8])], [1], 0.5, want_trace=True)   # keeps 2 of 4
            n, lo, hi = O.window(L, 0.5, 1, start, anchor)
            assert (n, hi - lo) == (2, 2)
            cache[fill] = ([orc.read_kv(l, 0, 8) for l in range(L)], r["trace"][0])
        none, copy, reco = cache[O.FILL_NONE][0], cache[O.FILL_COPY][0], cache[O.FILL_RECOMPUTE][0]
        for l in range(L):
            if lo <= l < hi:
                assert np.isnan(none[l][0]).all() and np.isnan(none[l][1]).all()
                if lo == 0:
                    assert not copy[l][0].any() and not copy[l][1].any()
                else:
                    assert np.array_equal(copy[l][0], copy[lo - 1][0])
                    assert np.array_equal(copy[l][1], copy[lo - 1][1])
                # recompute: layer l's own V projection of the carried hidden state
                x = cache[O.FILL_RECOMPUTE][1][l]
                a = O.rmsnorm(x, w["attn_norm"][l], shape.rms_eps)
                nq = shape.n_q_heads * shape.head_dim
                nkv = shape.n_kv_heads * shape.head_dim
                wv = w["wqkv"][l][nq + nkv:].double().numpy()
                assert np.abs(reco[l][1] - wv @ a).max() < 1e-12
                assert np.abs(cache[O.FILL_RECOMPUTE][1][l] - cache[O.FILL_RECOMPUTE][1][l + 1]).max() == 0
            else:
                for other in (copy, reco):
                    assert np.array_equal(none[l][0], other[l][0])
                    assert np.array_equal(none[l][1], other[l][1])


def test_batched_step_equals_rows_alone():
    shape = I.TINY
    w = I.make_weights(shape, SEED + 5, gain_jitter=0.1)
    L, alpha = shape.n_layers, 0.97
    prompts = [I.prompt_tokens(shape, SEED + 5, b, 5 + 3 * b) for b in range(4)]
    a = O.Oracle(shape, w, 4, 64, start_id=1)
    singles = [O.Oracle(shape, w, 1, 64, start_id=1) for _ in range(4)]
    for b in range(4):
        a.prefill(3 - b, prompts[b].numpy())
        singles[b].prefill(0, prompts[b].numpy())
    gi = [1, 30, 9, 55]
    for step in range(6):
        toks = [int(I.token_ids(SEED + 5, 900 + step, 4, shape.vocab)[b]) for b in range(4)]
        r = a.decode_step([3, 2, 1, 0], toks, [g + step for g in gi], alpha)
        for b in range(4):
            s = singles[b].decode_step([0], [toks[b]], [gi[b] + step], alpha)
            assert np.array_equal(r["logits"][b], s["logits"][0])


def test_error_paths():
    shape = I.TINY
    w = I.make_weights(shape, SEED, gain_jitter=0.0)
    orc = O.Oracle(shape, w, 2, 8)
    with pytest.raises(ValueError):
        orc.decode_step([0], [1], [1], 0.9)              # decode before prefill
    orc.prefill(0, [1, 2, 3])
    orc.prefill(1, [1, 2, 3])
    for bad in [dict(slots=[0, 0], tokens=[1, 1], gen_index=[1, 1], alpha=0.9),     # duplicate slot
                dict(slots=[0], tokens=[1], gen_index=[0], alpha=0.9),              # i < 1
                dict(slots=[0], tokens=[shape.vocab], gen_index=[1], alpha=0.9),    # token id
                dict(slots=[2], tokens=[1], gen_index=[1], alpha=0.9),              # slot
                dict(slots=[0], tokens=[1], gen_index=[1], alpha=1.5),
                dict(slots=[0], tokens=[1], gen_index=[1], alpha=float("nan"))]:
        with pytest.raises(ValueError):
            orc.decode_step(**bad)
    for i in range(5):
        orc.decode_step([0], [1], [i + 1], 0.9)
    with pytest.raises(ValueError):
        orc.decode_step([0], [1], [6], 0.9)              # cache full
    with pytest.raises(ValueError):
        O.Oracle(shape, w, 1, 8, start_id=5)


# ----------------------------------------------------------- textbook properties

def test_softmax_properties():
    p = O.softmax([0.0, math.log(3.0)])
    assert np.allclose(p, [0.25, 0.75], atol=1e-15)
    s = np.random.default_rng(0).normal(size=37) * 4
    p = O.softmax(s)
    assert abs(p.sum() - 1) < 1e-14 and (p > 0).all()
    assert np.allclose(p, O.softmax(s + 123.0), atol=1e-13)          # shift invariance
    assert np.isfinite(O.softmax([1000.0, -1000.0])).all()


def test_rmsnorm_closed_forms():
    g = torch.tensor([1.0, 2.0, 0.5, 1.0], dtype=torch.bfloat16)
    out = O.rmsnorm([3.0, 3.0, -3.0, 3.0], g, 0.0)
    assert np.allclose(out, [1.0, 2.0, -0.5, 1.0], atol=1e-15)
    out = O.rmsnorm([3.0, 3.0, -3.0, 3.0], g, 7.0)                    # eps inside the root
    assert np.allclose(out, np.array([3, 6, -1.5, 3]) / 4.0, atol=1e-15)
    assert not np.isnan(O.rmsnorm([0.0] * 4, g, 1e-5)).any()
    x = np.random.default_rng(1).normal(size=256)
    y = O.rmsnorm(x, torch.ones(256, dtype=torch.bfloat16), 0.0)
    assert abs(np.sqrt((y ** 2).mean()) - 1) < 1e-14


def test_rope_closed_forms():
    # dh = 2: one pair, theta_0 = 1, rotation by `pos` radians, counter-clockwise
    v = O.rope([1.0, 0.0], 1, 10000.0)
    assert np.allclose(v, [math.cos(1), math.sin(1)], atol=1e-15)
    v = O.rope([0.0, 1.0], 2, 10000.0)
    assert np.allclose(v, [-math.sin(2), math.cos(2)], atol=1e-15)
    # dh = 4: pairs (0,2) and (1,3); theta_1 = base^(-2/4)
    v = O.rope([1.0, 1.0, 0.0, 0.0], 3, 100.0)
    assert np.allclose(v, [math.cos(3), math.cos(0.3), math.sin(3), math.sin(0.3)], atol=1e-15)
    rng = np.random.default_rng(2)
    q, k = rng.normal(size=64), rng.normal(size=64)
    assert abs(np.linalg.norm(O.rope(q, 17, 1e4)) - np.linalg.norm(q)) < 1e-13
    d1 = O.rope(q, 9, 1e4) @ O.rope(k, 4, 1e4)
    d2 = O.rope(q, 25, 1e4) @ O.rope(k, 20, 1e4)
    assert abs(d1 - d2) < 1e-12                                       # depends on m - n only
    assert np.array_equal(O.rope(q, 0, 1e4), q)


def test_attention_special_cases():
    # d = 4, one head of dim 4, one block whose weights make the arithmetic visible
    shape = I.ModelShape("unit", 1, 4, 1, 1, 4, 4, 8)
    z = lambda *s: torch.zeros(*s, dtype=torch.bfloat16)
    eye = torch.eye(4, dtype=torch.bfloat16)
    emb = torch.tensor(np.random.default_rng(3).normal(size=(8, 4)), dtype=torch.bfloat16)
    w = {"embed": emb, "lm_head": torch.cat([eye, eye]), "final_norm": torch.ones(4, dtype=torch.bfloat16),
         "attn_norm": [torch.ones(4, dtype=torch.bfloat16)], "mlp_norm": [torch.ones(4, dtype=torch.bfloat16)],
         "wqkv": [torch.cat([z(4, 4), z(4, 4), eye])], "wo": [eye.clone()],
         "w_gate": [z(4, 4)], "w_up": [z(4, 4)], "w_down": [z(4, 4)]}
    # W_q = 0: uniform attention, so the block adds the mean of the normalised
    # embeddings seen so far; the MLP adds nothing (zero weights).
    orc = O.Oracle(shape, w, 1, 8)
    toks = [3, 5, 1, 6]
    _, hid = orc.prefill(0, toks, want_hidden=True)
    e = emb.double().numpy()
    a = np.stack([e[t] / math.sqrt((e[t] ** 2).mean() + shape.rms_eps) for t in toks])
    assert np.abs(hid - (e[6] + a.mean(axis=0))).max() < 1e-12
    r = orc.decode_step([0], [2], [1], 1.0)
    a2 = e[2] / math.sqrt((e[2] ** 2).mean() + shape.rms_eps)
    want = e[2] + (a.sum(axis=0) + a2) / 5
    assert np.abs(r["hidden"][0] - want).max() < 1e-12
    # zero W_o and W_down: the block is the identity on the residual stream
    w2 = dict(w)
    w2["wo"] = [z(4, 4)]
    orc2 = O.Oracle(shape, w2, 1, 8)
    _, hid2 = orc2.prefill(0, toks, want_hidden=True)
    assert np.array_equal(hid2, e[6])


def test_swiglu_closed_form():
    # attention switched off (W_o = 0); MLP: gate = 2 a_0, up = a_1, down = identity column
    shape = I.ModelShape("unit", 1, 2, 1, 1, 2, 1, 4)
    bf = lambda v: torch.tensor(v, dtype=torch.bfloat16)
    w = {"embed": bf([[1.0, 0.5], [0.25, -1.0], [2.0, 2.0], [-1.0, 0.5]]), "lm_head": bf([[1, 0], [0, 1], [1, 1], [1, -1]]),
         "final_norm": bf([1.0, 1.0]), "attn_norm": [bf([1.0, 1.0])], "mlp_norm": [bf([1.0, 1.0])],
         "wqkv": [torch.zeros(6, 2, dtype=torch.bfloat16)], "wo": [torch.zeros(2, 2, dtype=torch.bfloat16)],
         "w_gate": [bf([[2.0, 0.0]])], "w_up": [bf([[0.0, 1.0]])], "w_down": [bf([[0.0], [1.0]])]}
    orc = O.Oracle(shape, w, 1, 4)
    for tok in range(4):
        _, hid = orc.prefill(0, [tok], want_hidden=True)
        x = w["embed"][tok].double().numpy()
        a = x / math.sqrt((x ** 2).mean() + shape.rms_eps)
        g = 2 * a[0]
        want = x + np.array([0.0, g / (1 + math.exp(-g)) * a[1]])
        assert np.abs(hid - want).max() < 1e-14


def test_fp32_build_tracks_fp64():
    shape = I.TINY_GQA
    w = I.make_weights(shape, SEED + 6, gain_jitter=0.1)
    toks = I.prompt_tokens(shape, SEED + 6, 0, 24)
    a = O.Oracle(shape, w, 1, 32, start_id=1)
    b = O.Oracle(shape, w, 1, 32, start_id=1, real="f32")
    la, lb = a.prefill(0, toks[:8].numpy()), b.prefill(0, toks[:8].numpy())
    assert np.abs(la - lb).max() < 2e-5
    for i in range(1, 16):
        ra = a.decode_step([0], [int(toks[7 + i])], [i], 0.93)
        rb = b.decode_step([0], [int(toks[7 + i])], [i], 0.93)
        assert np.abs(ra["logits"] - rb["logits"]).max() < 2e-5
