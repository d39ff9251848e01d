"""Parity of the CUDA path with the CPU oracle, through the C ABI (GPU)."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2503_08524_b200 import inputs as I

from parity import LOGITS_MAX_ABS, check_step, make_pair, rel_l2

pytestmark = pytest.mark.gpu
SEED = I.BASE_SEED


@pytest.fixture(scope="module")
def B():
    from paper_2503_08524_b200 import binding
    assert torch.cuda.is_available()
    return binding


# ------------------------------------------------------------ depth schedule (K0)

@pytest.mark.parametrize("anchor", [0, 1])
def test_schedule_kernel_is_bit_exact(B, anchor):
    shape = I.TINY
    rng = np.random.default_rng(3)
    for start, alpha in [(0, 0.95), (1, 0.98), (2, 0.9), (0, 1.0), (4, 0.5)]:
        orc, gpu = make_pair(shape, SEED, 64, 8, 64, start_id=start, anchor=anchor, kv_fill=0)
        for s in range(64):
            gpu.d3_prefill(s, [1, 2])
        for Bn in (1, 2, 3, 17, 64):
            gi = rng.integers(1, 60, size=Bn).astype(np.int32)
            gi[Bn // 2] = gi[0]
            slots = rng.permutation(64)[:Bn]
            _, st = gpu.d3_decode_step(slots, [5] * Bn, gi, alpha, want_stats=True)
            dev = gpu.d3_read_schedule(Bn)
            want = O.schedule(shape.n_layers, alpha, start, anchor, gi)
            host = B.d3_schedule(shape.n_layers, alpha, start, anchor, gi)
            for k in ("n", "perm", "m_per_layer"):
                assert np.array_equal(dev[k], want[k]), (k, Bn, start, alpha)
                assert np.array_equal(host[k], want[k])
            assert np.array_equal(st["n"], want["n"]) and np.array_equal(st["m_per_layer"], want["m_per_layer"])
            for k in ("rows_layers", "layers_touched"):
                assert dev[k] == want[k] == st[k]
            for s in slots:
                gpu.d3_reset_slot(int(s))
                gpu.d3_prefill(int(s), [1, 2])
        gpu.close()


def test_schedule_kernel_large_L(B):
    # 7B/13B/70B layer counts on a narrow model: only the integers matter here
    for L, alpha, start in [(32, 0.997, 6), (40, 0.998, 8), (80, 0.998, 16), (128, 0.99, 25)]:
        shape = I.ModelShape("narrow", L, 64, 2, 1, 32, 64, 128)
        orc, gpu = make_pair(shape, SEED, 32, 4, 32, start_id=start, kv_fill=1)
        for s in range(32):
            gpu.d3_prefill(s, [3])
        gi = np.array([1 + (8 * b) % 256 for b in range(32)], np.int32)
        gpu.d3_decode_step(list(range(32)), [7] * 32, gi, alpha)
        dev = gpu.d3_read_schedule(32)
        want = O.schedule(L, alpha, start, 0, gi)
        for k in ("n", "perm", "m_per_layer"):
            assert np.array_equal(dev[k], want[k]), (k, L)
        assert dev["rows_layers"] == want["rows_layers"] and dev["layers_touched"] == want["layers_touched"]
        gpu.close()


# --------------------------------------------------- tiny config, batch 1, whole run

@pytest.mark.parametrize("shape", [I.TINY, I.TINY_GQA], ids=["mha", "gqa"])
@pytest.mark.parametrize("alpha", [1.0, 0.98, 0.95])
@pytest.mark.parametrize("kv_round", [False, True], ids=["kv-exact", "kv-bf16"])
@pytest.mark.parametrize("exec_mode", [0, 1, 2], ids=["fused", "kernels", "tensor"])
def test_tiny_generate_teacher_forced(B, shape, alpha, kv_round, exec_mode):
    orc, gpu = make_pair(shape, SEED, 2, 64, 1, start_id=0, kv_round_bf16=kv_round)
    gpu.d3_set_exec(exec_mode)
    prompt = I.prompt_tokens(shape, SEED, 0, 16).numpy()
    o_lg, o_hid = orc.prefill(1, prompt, want_hidden=True)
    g_lg = gpu.d3_prefill(1, prompt)
    check_step("prefill", g_lg.cpu().numpy()[None], gpu.d3_read_hidden(1)[-1:], o_lg[None], o_hid[None])
    tok = O.argmax(o_lg)
    layers = 0
    for i in range(1, 32):
        r = orc.decode_step([1], [tok], [i], alpha)
        g, st = gpu.d3_decode_step([1], [tok], [i], alpha, want_stats=True)
        check_step(f"step {i}", g.cpu().numpy(), gpu.d3_read_hidden(1), r["logits"], r["hidden"])
        assert st["n"][0] == O.window(shape.n_layers, alpha, i, 0)[0]
        layers += st["rows_layers"]
        tok = O.argmax(r["logits"][0])
    gpu.d3_sync()
    assert layers == sum(O.depth(shape.n_layers, alpha, i) for i in range(1, 32))
    assert gpu.d3_slot_pos(1) == orc.slot_pos(1) == 16 + 31
    gpu.close()


def test_tiny_greedy_tokens_identical(B):
    # free-running greedy decode, argmax on the device, fed back on the device
    shape = I.TINY
    for alpha in (1.0, 0.98, 0.95):
        orc, gpu = make_pair(shape, SEED + 1, 1, 64, 1, gain_jitter=0.0, kv_round_bf16=False)
        prompt = I.prompt_tokens(shape, SEED + 1, 0, 16).numpy()
        o_tok = [O.argmax(orc.prefill(0, prompt))]
        margins = []
        for i in range(1, 32):
            lg = orc.decode_step([0], [o_tok[-1]], [i], alpha)["logits"][0]
            top = np.sort(lg)[-2:]
            margins.append(top[1] - top[0])
            o_tok.append(O.argmax(lg))
        lg = gpu.d3_prefill(0, prompt)
        tok = gpu.d3_argmax(lg)
        g_tok = [int(tok.item())]
        for i in range(1, 32):
            lg = gpu.d3_decode_step([0], None, [i], alpha, tokens_dev=tok)
            tok = gpu.d3_argmax(lg)
            g_tok.append(int(tok.item()))
        if min(margins) > 4 * LOGITS_MAX_ABS:
            assert g_tok == o_tok, alpha
        else:   # a near-tie may legitimately flip: compare up to the first such step
            k = next(j for j, m in enumerate(margins) if m <= 4 * LOGITS_MAX_ABS) + 1
            assert g_tok[:k] == o_tok[:k], alpha
        gpu.close()


# ------------------------------------------------ mixed-depth batches, anchors, fills

@pytest.mark.parametrize("anchor,start", [(0, 0), (0, 1), (0, 2), (1, 0)])
@pytest.mark.parametrize("fill", [0, 1, 2])
@pytest.mark.parametrize("exec_mode,paged", [(0, False), (1, False), (0, True)],
                         ids=["tensor-cores", "fma", "paged-kv"])
def test_batched_mixed_depth_steps(B, anchor, start, fill, exec_mode, paged):
    # exec 0: depth groups of 2+ rows project on the tensor cores, single rows by FMA GEMV;
    # exec 1: FMA GEMVs throughout; paged: the cache is a pool of 16-position pages
    shape = I.TINY_GQA
    Bn, alpha = 7, 0.96
    pk = dict(page_size=16, n_pages=1 + shape.n_layers * 8 * 6) if paged else {}
    orc, gpu = make_pair(shape, SEED + 2, 8, 96, 8, start_id=start, anchor=anchor, kv_fill=fill, **pk)
    gpu.d3_set_exec(exec_mode)
    gpu.poison_kv()
    orc.poison_kv()
    lens = I.uniform_ints(SEED + 2, 77, Bn, 3, 40)
    slots = [5, 0, 7, 2, 3, 6, 1]
    for b in range(Bn):
        p = I.prompt_tokens(shape, SEED + 2, b, lens[b]).numpy()
        o = orc.prefill(slots[b], p)
        g = gpu.d3_prefill(slots[b], p)
        check_step(f"prefill {b}", g.cpu().numpy()[None], None, o[None], None)
    gi0 = [1, 9, 30, 2, 55, 17, 9]
    seen = set()
    for step in range(12):
        toks = I.token_ids(SEED + 2, 500 + step, Bn, shape.vocab).numpy()
        gi = [g + step for g in gi0]
        r = orc.decode_step(slots, toks, gi, alpha)
        g, st = gpu.d3_decode_step(slots, toks, gi, alpha, want_stats=True)
        check_step(f"step {step}", g.cpu().numpy(), gpu.d3_read_hidden(Bn), r["logits"], r["hidden"])
        seen.update(int(v) for v in st["n"])
    assert len(seen) >= 2
    # the caches agree wherever the oracle holds a number (bf16 storage on the GPU)
    for b in range(Bn):
        pos = orc.slot_pos(slots[b]) - 1
        for l in range(shape.n_layers):
            ok, ov = orc.read_kv(l, slots[b], pos)
            gk, gv = gpu.d3_read_kv(l, slots[b], pos)
            if np.isnan(ok).any():
                assert np.isnan(gk).all() and np.isnan(gv).all()      # FILL_NONE leaves it alone
            else:
                assert np.abs(gk - ok).max() <= 0.02 * max(1.0, np.abs(ok).max())
                assert np.abs(gv - ov).max() <= 0.02 * max(1.0, np.abs(ov).max())
    gpu.close()


@pytest.mark.parametrize("anchor,start", [(0, 0), (0, 1), (0, 3), (1, 0)])
@pytest.mark.parametrize("fill", [0, 1])
def test_fused_step_fills_and_long_context(B, anchor, start, fill):
    # batch 1 through the single-kernel step: several KV chunks per head (the
    # last one ragged), windows at both anchors, cache contents against the oracle
    shape = I.TINY_GQA
    orc, gpu = make_pair(shape, SEED + 7, 1, 700, 16, start_id=start, anchor=anchor, kv_fill=fill)
    gpu.poison_kv()
    orc.poison_kv()
    prompt = I.prompt_tokens(shape, SEED + 7, 0, 389).numpy()
    o = orc.prefill(0, prompt)
    g = gpu.d3_prefill(0, prompt)
    check_step("prefill", g.cpu().numpy()[None], None, o[None], None)
    toks = I.token_ids(SEED + 7, 5, 40, shape.vocab).numpy()
    for i in range(1, 30):
        r = orc.decode_step([0], [int(toks[i])], [i], 0.93)
        g, st = gpu.d3_decode_step([0], [int(toks[i])], [i], 0.93, want_stats=True)
        assert st["kernel_launches"] == 1
        check_step(f"step {i}", g.cpu().numpy(), gpu.d3_read_hidden(1), r["logits"], r["hidden"])
        dev = gpu.d3_read_schedule(1)
        want = O.schedule(shape.n_layers, 0.93, start, anchor, [i])
        assert np.array_equal(dev["n"], want["n"]) and np.array_equal(dev["m_per_layer"], want["m_per_layer"])
        pos = orc.slot_pos(0) - 1
        for l in range(shape.n_layers):
            ok, ov = orc.read_kv(l, 0, pos)
            gk, gv = gpu.d3_read_kv(l, 0, pos)
            if np.isnan(ok).any():
                assert np.isnan(gk).all() and np.isnan(gv).all()
            else:
                assert np.abs(gk - ok).max() <= 0.02 * max(1.0, np.abs(ok).max())
                assert np.abs(gv - ov).max() <= 0.02 * max(1.0, np.abs(ov).max())
    gpu.d3_sync()
    gpu.close()


@pytest.mark.parametrize("fill", [1, 2])
def test_alpha_raised_mid_sequence_reads_filled_entries(B, fill):
    # depth grows again when the caller raises alpha: later tokens then read what
    # the fill mode left in the cache (defined by the fill rule only)
    shape = I.TINY
    orc, gpu = make_pair(shape, SEED + 3, 1, 64, 1, start_id=1, kv_fill=fill)
    prompt = I.prompt_tokens(shape, SEED + 3, 0, 8).numpy()
    tok = O.argmax(orc.prefill(0, prompt))
    gpu.d3_prefill(0, prompt)
    for i in range(1, 24):
        alpha = 0.9 if i < 12 else 1.0
        r = orc.decode_step([0], [tok], [i], alpha)
        g = gpu.d3_decode_step([0], [tok], [i], alpha)
        check_step(f"step {i}", g.cpu().numpy(), gpu.d3_read_hidden(1), r["logits"], r["hidden"])
        tok = O.argmax(r["logits"][0])
    gpu.close()


def test_prefill_longer_than_a_batch_and_ragged_lengths(B):
    shape = I.TINY
    orc, gpu = make_pair(shape, SEED + 4, 3, 200, 16)
    for slot, n in [(0, 1), (1, 16), (2, 17), (0, 131)]:
        p = I.prompt_tokens(shape, SEED + 4, slot + n, n).numpy()
        o, oh = orc.prefill(slot, p, want_hidden=True)
        g = gpu.d3_prefill(slot, p)
        check_step(f"prefill {n}", g.cpu().numpy()[None], None, o[None], None)
        assert gpu.d3_slot_pos(slot) == n
    # long context decode: several attention splits with a ragged tail
    tok = 3
    for i in range(1, 6):
        r = orc.decode_step([0, 2], [tok, tok], [i, i + 3], 0.97)
        g = gpu.d3_decode_step([0, 2], [tok, tok], [i, i + 3], 0.97)
        check_step(f"step {i}", g.cpu().numpy(), gpu.d3_read_hidden(2), r["logits"], r["hidden"])
    gpu.close()


# ----------------------------------------------------------- production widths

@pytest.mark.parametrize("base,layers,Bn", [(I.LLAMA_7B, 3, 1), (I.LLAMA_7B, 2, 5), (I.LLAMA_70B, 2, 3),
                                            (I.LLAMA_13B, 2, 1), (I.LLAMA_70B, 2, 1), (I.LLAMA_7B, 2, 32),
                                            (I.LLAMA_13B, 2, 8), (I.LLAMA_70B, 2, 4), (I.LLAMA_7B, 2, -5)],
                         ids=["7b-width-b1", "7b-width-b5", "70b-width-gqa-b3", "13b-width-b1",
                              "70b-width-gqa-b1", "7b-width-b32", "13b-width-b8", "70b-width-gqa-b4",
                              "7b-width-b5-paged-kv"])
def test_production_widths(B, base, layers, Bn):
    # full-width blocks (same kernel shapes and tiling as the benchmark), few layers;
    # batches of 2+ rows take the tensor-core projections, single rows the fused step
    shape = base.with_layers(layers)
    pk = {}
    if Bn < 0:      # negative row count: the same case over a paged cache (32-position pages)
        Bn = -Bn
        pk = dict(page_size=32, n_pages=1 + layers * Bn * 3)
    orc, gpu = make_pair(shape, SEED + 5, Bn, 96, max(8, Bn), start_id=1, gain_jitter=0.1, **pk)
    lens = I.uniform_ints(SEED + 5, 3, Bn, 5, 40 if Bn <= 8 else 12)
    for b in range(Bn):
        p = I.prompt_tokens(shape, SEED + 5, b, lens[b]).numpy()
        o = orc.prefill(b, p)
        g = gpu.d3_prefill(b, p)
        check_step(f"prefill {b}", g.cpu().numpy()[None], None, o[None], None)
    for step in range(4):
        # single rows: the single-kernel step on even steps, the tensor-core kernel sequence on odd ones
        gpu.d3_set_exec((B.EXEC_AUTO if step % 2 == 0 else B.EXEC_TENSOR) if (Bn == 1 and not pk) else B.EXEC_AUTO)
        toks = I.token_ids(SEED + 5, 40 + step, Bn, shape.vocab).numpy()
        gi = [1 + step + 2 * b for b in range(Bn)]
        alpha = 0.8
        r = orc.decode_step(list(range(Bn)), toks, gi, alpha)
        g, st = gpu.d3_decode_step(list(range(Bn)), toks, gi, alpha, want_stats=True)
        check_step(f"step {step}", g.cpu().numpy(), gpu.d3_read_hidden(Bn), r["logits"], r["hidden"])
        if Bn == 1 and not pk and step % 2 == 0:
            assert st["kernel_launches"] == 1
    gpu.d3_sync()          # raises on a deferred device status (a bounded wait that ran out)
    gpu.close()


def test_thirty_two_rows_at_7b_width_with_long_and_short_contexts(B):
    """The batched workload's own step shape: 7B-width blocks, 32 rows in one step, contexts from a
    few tokens up to 1024 (the attention pass then cuts the long rows into pieces and merges them),
    retained depths mixed inside the step.  Two blocks keep the oracle's prefill of the long rows
    to about half a minute."""
    shape = I.LLAMA_7B.with_layers(2)
    Bn = 32
    orc, gpu = make_pair(shape, SEED + 21, Bn, 1040, Bn, start_id=1, kv_fill=1)
    long_rows = {0: 1024, 5: 640, 11: 300, 18: 128, 31: 513}
    short = I.uniform_ints(SEED + 21, 2, Bn, 3, 12)
    for b in range(Bn):
        n = long_rows.get(b, int(short[b]))
        p = I.prompt_tokens(shape, SEED + 21, b, n).numpy()
        o = orc.prefill(b, p)
        g = gpu.d3_prefill(b, p)
        if b in long_rows:
            check_step(f"prefill {b}", g.cpu().numpy()[None], None, o[None], None)
    for step in range(2):
        toks = I.token_ids(SEED + 21, 50 + step, Bn, shape.vocab).numpy()
        depths = [2 if (b + step) % 3 else 1 for b in range(Bn)]   # long rows on both sides of the cut
        r = orc.decode_step_depths(list(range(Bn)), toks, depths)
        g, st = gpu.d3_decode_step_depths(list(range(Bn)), toks, depths, want_stats=True)
        check_step(f"step {step}", g.cpu().numpy(), gpu.d3_read_hidden(Bn), r["logits"], r["hidden"])
        assert st["rows_layers"] == sum(depths)
    gpu.d3_sync()
    gpu.close()


# ------------------------------------------------ the largest step the ABI allows

def test_sixty_four_rows_per_step(B):
    # D3_MAX_BATCH rows: the widest tensor-core operand (3 x 64 rows -> UMMA N = 192, 256 TMEM
    # columns, two-stage ring), 64-position prefill passes, every depth from L - 1 down to 0 in one step
    shape = I.TINY_GQA
    Bn, L = 64, shape.n_layers
    orc, gpu = make_pair(shape, SEED + 14, Bn, 160, Bn, start_id=0, kv_fill=1)
    for b in range(Bn):
        n = 1 + (37 * b) % 90                      # 1 .. 90 tokens: one or two passes, ragged
        p = I.prompt_tokens(shape, SEED + 14, b, n).numpy()
        o = orc.prefill(b, p)
        g = gpu.d3_prefill(b, p)
        if b % 8 == 0:
            check_step(f"prefill {b}", g.cpu().numpy()[None], None, o[None], None)
    seen = set()
    for step in range(3):
        toks = I.token_ids(SEED + 14, 70 + step, Bn, shape.vocab).numpy()
        gi = [1 + step + b for b in range(Bn)]
        r = orc.decode_step(list(range(Bn)), toks, gi, 0.955)
        g, st = gpu.d3_decode_step(list(range(Bn)), toks, gi, 0.955, want_stats=True)
        check_step(f"step {step}", g.cpu().numpy(), gpu.d3_read_hidden(Bn), r["logits"], r["hidden"])
        want = O.schedule(L, 0.955, 0, 0, gi)
        assert np.array_equal(st["n"], want["n"]) and np.array_equal(st["m_per_layer"], want["m_per_layer"])
        seen.update(int(v) for v in st["n"])
    assert seen == set(range(L))                    # floor(4 * 0.955^i): 3 down to 0
    with pytest.raises(B.D3Error) as e:             # 65 rows: over the limit of the model
        gpu.d3_decode_step(list(range(Bn)) + [0], [1] * 65, [1] * 65, 1.0)
    assert e.value.code == B.ECAPACITY
    gpu.d3_sync()
    gpu.close()


# ------------------------------------------------ tensor-core attention, every variant

@pytest.mark.parametrize("hq,hkv,dh", [(32, 32, 128), (32, 32, 64), (32, 16, 128), (32, 8, 32), (16, 4, 64),
                                       (32, 32, 32)],
                         ids=["mha-128", "mha-64", "gq2-128", "gq4-32", "gq4-64", "mha-32"])
def test_tensor_core_attention_variants(B, hq, hkv, dh):
    # Many heads on a narrow model: rows x heads exceeds the CTA target, so every (row, head group)
    # takes ONE piece of 260-340 positions (several 16-position trips per warp, a ragged last
    # trip) and the MHA variants take the tensor-core kernel too (it needs >= 256 positions per
    # piece there).  Contexts differ per row; 20 rows; against the oracle.
    shape = I.ModelShape(f"heads-{hq}-{hkv}-{dh}", 2, 256, hq, hkv, dh, 512, 1024)
    Bn = 20
    orc, gpu = make_pair(shape, SEED + 15, Bn, 352, 32, start_id=0)
    lens = I.uniform_ints(SEED + 15, 2, Bn, 260, 335)
    for b in range(Bn):
        p = I.prompt_tokens(shape, SEED + 15, b, lens[b]).numpy()
        o = orc.prefill(b, p)
        g = gpu.d3_prefill(b, p)
        if b % 5 == 0:
            check_step(f"prefill {b}", g.cpu().numpy()[None], None, o[None], None)
    for step in range(3):
        toks = I.token_ids(SEED + 15, 20 + step, Bn, shape.vocab).numpy()
        gi = [1 + step + b for b in range(Bn)]
        r = orc.decode_step(list(range(Bn)), toks, gi, 0.97)
        g = gpu.d3_decode_step(list(range(Bn)), toks, gi, 0.97)
        check_step(f"step {step}", g.cpu().numpy(), gpu.d3_read_hidden(Bn), r["logits"], r["hidden"])
    gpu.d3_sync()
    gpu.close()


# ------------------------------------------------ depths given by the caller

@pytest.mark.parametrize("anchor,start,fill", [(0, 1, 1), (0, 0, 0), (1, 0, 2)])
def test_steps_with_given_depths_linear_decay(B, anchor, start, fill):
    # d3_decode_step_depths: the retained count of every row comes from the caller, here from the
    # linear-decay rule (Sec. 3.4 / 4.1).  A batch of 5 rows at staggered indices (sequence of
    # kernels, tensor-core projections) and a single row (single-kernel step), against the oracle.
    shape = I.TINY_GQA
    L, Bn = shape.n_layers, 5
    orc, gpu = make_pair(shape, SEED + 12, 6, 96, 8, start_id=start, anchor=anchor, kv_fill=fill)
    lens = I.uniform_ints(SEED + 12, 1, Bn + 1, 3, 30)
    for b in range(Bn + 1):
        p = I.prompt_tokens(shape, SEED + 12, b, lens[b]).numpy()
        orc.prefill(b, p)
        gpu.d3_prefill(b, p)
    seen = set()
    for step in range(14):
        depths = [O.depth_linear(L, 1, 12, 1 + step + 3 * b) for b in range(Bn)]
        assert depths == [B.d3_depth_linear(L, 1, 12, 1 + step + 3 * b) for b in range(Bn)]
        toks = I.token_ids(SEED + 12, 300 + step, Bn + 1, shape.vocab).numpy()
        r = orc.decode_step_depths(list(range(Bn)), toks[:Bn], depths)
        g, st = gpu.d3_decode_step_depths(list(range(Bn)), toks[:Bn], depths, want_stats=True)
        check_step(f"batch step {step}", g.cpu().numpy(), gpu.d3_read_hidden(Bn), r["logits"], r["hidden"])
        want = [O.window_of_depth(L, d, start, anchor)[0] for d in depths]
        assert list(st["n"]) == want and st["rows_layers"] == sum(want)
        dev = gpu.d3_read_schedule(Bn)
        assert list(dev["n"]) == want                     # the device derived the same counts
        seen.update(want)
        # one row alone: the single-kernel step (fill RECOMPUTE runs the kernel sequence)
        d1 = O.depth_linear(L, 0, 9, step)
        r1 = orc.decode_step_depths([Bn], [int(toks[Bn])], [d1])
        g1, st1 = gpu.d3_decode_step_depths([Bn], [int(toks[Bn])], [d1], want_stats=True)
        check_step(f"single step {step}", g1.cpu().numpy(), gpu.d3_read_hidden(1), r1["logits"], r1["hidden"])
        assert st1["kernel_launches"] == 1 or fill == 2
    assert len(seen) >= 3
    for bad in ([L + 1], [-1]):
        with pytest.raises(B.D3Error) as e:
            gpu.d3_decode_step_depths([0], [1], bad)
        assert e.value.code == B.EINVAL
    gpu.d3_sync()
    gpu.close()


# ------------------------------------------------ saturation probe

@pytest.mark.parametrize("shape,Bn", [(I.TINY, 3), (I.TINY_GQA, 1)], ids=["mha-b3", "gqa-b1"])
def test_saturation_probe_matches_oracle(B, shape, Bn):
    # Sec. 3.2: per block, the token and confidence the LM head predicts from the block's output
    L = shape.n_layers
    orc, gpu = make_pair(shape, SEED + 13, Bn, 64, 4)
    for b in range(Bn):
        p = I.prompt_tokens(shape, SEED + 13, b, 5 + 4 * b).numpy()
        orc.prefill(b, p)
        gpu.d3_prefill(b, p)
    for step in range(3):
        toks = I.token_ids(SEED + 13, 50 + step, Bn, shape.vocab).numpy()
        r = orc.saturation_probe(list(range(Bn)), toks)
        lg, gt, gc = gpu.d3_saturation_probe(list(range(Bn)), toks)
        check_step(f"step {step}", lg.cpu().numpy(), gpu.d3_read_hidden(Bn), r["logits"], r["hidden"])
        gt, gc = gt.cpu().numpy(), gc.cpu().numpy()
        for b in range(Bn):
            assert gpu.d3_slot_pos(b) == orc.slot_pos(b)
            for i in range(1, L + 1):
                _, _, ol = orc.probe(r["trace"][b, i])
                top = np.sort(ol)[-2:]
                if top[1] - top[0] > 4 * LOGITS_MAX_ABS:          # not a near-tie
                    assert gt[b, i - 1] == r["tokens"][b, i - 1], (b, i)
                    assert abs(gc[b, i - 1] - r["conf"][b, i - 1]) <= 0.05 * r["conf"][b, i - 1] + 1e-6
                else:                                              # either candidate is valid
                    assert ol[gt[b, i - 1]] >= top[1] - 4 * LOGITS_MAX_ABS
            assert gt[b, L - 1] == int(gpu.d3_argmax(lg)[b].item())
    gpu.d3_sync()
    gpu.close()


# ------------------------------------------------ the benchmark model at full depth

def test_full_depth_7b_shape_against_oracle_and_between_paths(B):
    # All 32 blocks of the 7B shape, batch 1, decode in the launch configuration the benchmark
    # times (single-kernel step), teacher-forced, at generation indices on both sides of depth
    # transitions of alpha = 0.995.
    # (a) Oracle parity on a 32-token prompt.  The cache is bf16 on both sides, so a K or V
    #     element rounds differently wherever the two sides' fp values straddle a rounding
    #     boundary; how often depends on the error of the arithmetic that produced them.  The
    #     prompt is projected once by the fp32-FMA kernels and once by the tensor-core kernels
    #     (whose K and V rows are summed in short chains for this reason); both runs are held to
    #     the stated tolerances.
    # (b) At the benchmark's prompt length (512), also a property: the single-kernel step and the
    #     sequence of kernels (independent implementations) agree on the same steps.  (The oracle
    #     comparison at that length is the next test.)
    shape, alpha, start = I.LLAMA_7B, 0.995, 6
    L = shape.n_layers
    orc, gpu = make_pair(shape, SEED + 11, 1, 600, 32, start_id=start, gain_jitter=0.0)
    prompt = I.prompt_tokens(shape, SEED + 11, 0, 32).numpy()
    gis = [1, 6, 7, 12, 13, 138, 139, 255]
    assert O.depth(L, alpha, 6) == 31 and O.depth(L, alpha, 7) == 30
    assert O.depth(L, alpha, 138) == 16 and O.depth(L, alpha, 139) == 15
    toks = I.token_ids(SEED + 11, 9, len(gis), shape.vocab).numpy()
    o_pre = orc.prefill(0, prompt)
    ref = [orc.decode_step([0], [int(toks[k])], [i], alpha) for k, i in enumerate(gis)]
    orc.close()
    for prefill_exec, logit_tol in ((B.EXEC_KERNELS, LOGITS_MAX_ABS), (B.EXEC_AUTO, LOGITS_MAX_ABS)):
        gpu.d3_set_exec(prefill_exec)
        gpu.d3_reset_slot(0)
        g = gpu.d3_prefill(0, prompt).cpu().numpy()
        assert np.isfinite(g).all() and np.abs(g - o_pre).max() <= logit_tol, prefill_exec
        gpu.d3_set_exec(B.EXEC_AUTO)
        for k, i in enumerate(gis):
            gl, st = gpu.d3_decode_step([0], [int(toks[k])], [i], alpha, want_stats=True)
            assert st["kernel_launches"] == 1 and st["n"][0] == max(O.depth(L, alpha, i), start)
            gl = gl.cpu().numpy()
            assert np.isfinite(gl).all()
            assert np.abs(gl - ref[k]["logits"]).max() <= logit_tol, (prefill_exec, i)
            assert rel_l2(gpu.d3_read_hidden(1)[0], ref[k]["hidden"][0]) <= 1e-2, (prefill_exec, i)
    # (b) benchmark prompt length: both GPU paths, same steps
    prompt = I.prompt_tokens(shape, SEED + 11, 1, 512).numpy()
    outs = {}
    for mode in (B.EXEC_AUTO, B.EXEC_KERNELS):
        gpu.d3_set_exec(B.EXEC_AUTO)
        gpu.d3_reset_slot(0)
        gpu.d3_prefill(0, prompt)
        gpu.d3_set_exec(mode)
        res = []
        for k, i in enumerate(gis):
            gl = gpu.d3_decode_step([0], [int(toks[k])], [i], alpha)
            res.append((gl.cpu().numpy().copy(), gpu.d3_read_hidden(1).copy()))
        outs[mode] = res
    for k, i in enumerate(gis):
        (l0, h0), (l1, h1) = outs[B.EXEC_AUTO][k], outs[B.EXEC_KERNELS][k]
        assert np.isfinite(l0).all() and np.abs(l0 - l1).max() <= LOGITS_MAX_ABS, i
        assert rel_l2(h0[0], h1[0]) <= 1e-2, i
    gpu.d3_sync()
    gpu.close()


def test_benchmark_configuration_against_the_oracle(B):
    # The benchmark's own configuration against the oracle: 7B shape, all 32 blocks, batch 1,
    # prompt of 512 tokens through the batched prefill (passes of 128 positions, as bench.py loads
    # the model), then single-kernel decode steps at alpha = 0.995 on both sides of the depth
    # transition 31 -> 30 and at depth 15, teacher-forced.  The oracle's 512-token prefill takes a
    # minute or two of CPU time.
    shape, alpha, start, P = I.LLAMA_7B, 0.995, 6, 512
    L = shape.n_layers
    orc, gpu = make_pair(shape, SEED + 17, 1, P + 8, 128, start_id=start, gain_jitter=0.0)
    prompt = I.prompt_tokens(shape, SEED + 17, 0, P).numpy()
    gis = [6, 7, 139]
    toks = I.token_ids(SEED + 17, 9, len(gis), shape.vocab).numpy()
    o_pre, o_hid = orc.prefill(0, prompt, want_hidden=True)
    g = gpu.d3_prefill(0, prompt).cpu().numpy()
    assert np.isfinite(g).all()
    assert np.abs(g - o_pre).max() <= LOGITS_MAX_ABS, np.abs(g - o_pre).max()
    assert rel_l2(gpu.d3_read_hidden(128)[(P - 1) % 128], o_hid) <= 1e-2
    for k, i in enumerate(gis):
        r = orc.decode_step([0], [int(toks[k])], [i], alpha)
        gl, st = gpu.d3_decode_step([0], [int(toks[k])], [i], alpha, want_stats=True)
        assert st["kernel_launches"] == 1 and st["n"][0] == max(O.depth(L, alpha, i), start)
        check_step(f"i={i}", gl.cpu().numpy(), gpu.d3_read_hidden(1), r["logits"], r["hidden"])
    gpu.d3_sync()
    gpu.close()
    orc.close()


# ------------------------------------------------------------------ paged KV cache

def test_paged_cache_single_row_run_and_page_accounting(B):
    # batch 1 over a paged cache, depth decaying over page boundaries.
    # FILL_NONE never writes a dropped (token, block) pair, so a block stops taking pages once
    # the tokens stop running it; FILL_COPY writes every pair and takes pages like a dense cache.
    shape = I.TINY
    L, ps, alpha, start = shape.n_layers, 16, 0.93, 1
    used = {}
    for fill in (0, 1):
        orc, gpu = make_pair(shape, SEED + 9, 2, 96, 4, start_id=start, kv_fill=fill, page_size=ps,
                             n_pages=1 + 2 * L * 6)
        gpu.poison_kv()
        orc.poison_kv()
        prompt = I.prompt_tokens(shape, SEED + 9, 0, 21).numpy()
        o = orc.prefill(0, prompt)
        g = gpu.d3_prefill(0, prompt)
        check_step("prefill", g.cpu().numpy()[None], None, o[None], None)
        assert gpu.d3_kv_pages_used() == L * 2                      # positions 0..20: two pages per block
        written = {(l, p // ps) for l in range(L) for p in range(21)}
        toks = I.token_ids(SEED + 9, 5, 64, shape.vocab).numpy()
        for i in range(1, 50):
            pos = orc.slot_pos(0)
            r = orc.decode_step([0], [int(toks[i])], [i], alpha)
            g = gpu.d3_decode_step([0], [int(toks[i])], [i], alpha)
            check_step(f"step {i}", g.cpu().numpy(), gpu.d3_read_hidden(1), r["logits"], r["hidden"])
            n, lo, hi = O.window(L, alpha, i, start)
            for l in range(L):
                if fill != 0 or not (lo <= l < hi):
                    written.add((l, pos // ps))
            assert gpu.d3_kv_pages_used() == len(written), (fill, i)
        used[fill] = gpu.d3_kv_pages_used()
        # a second sequence takes its own pages; resetting it gives exactly those back
        gpu.d3_prefill(1, prompt[:5])
        assert gpu.d3_kv_pages_used() == used[fill] + L
        gpu.d3_reset_slot(1)
        assert gpu.d3_kv_pages_used() == used[fill]
        gpu.d3_sync()
        gpu.close()
    assert used[1] == L * 5                                          # 70 positions, dense
    assert used[0] < used[1]                                         # the depth-aware saving


@pytest.mark.parametrize("shape,ps,fill", [(I.TINY, 16, 1), (I.TINY, 64, 0), (I.TINY, 128, 1), (I.TINY_GQA, 16, 1),
                                           (I.TINY_GQA, 256, 0), (I.LLAMA_7B.with_layers(2), 16, 1),
                                           (I.LLAMA_7B.with_layers(2), 32, 1)],
                         ids=["dh64-p16", "dh64-p64-none", "dh64-p128", "dh32-gqa-p16", "dh32-gqa-p256-none",
                              "7b-width-p16", "7b-width-p32"])
def test_single_kernel_step_over_a_paged_cache(B, shape, ps, fill):
    # One row over a paged cache takes the single-kernel step like a contiguous model: its
    # producers fetch a ring stage of K and V as one run per page (pages shorter than a stage:
    # several runs), the tail positions and the appended / filled entries go through the page table.
    L = shape.n_layers
    wide = shape.d_model > 1024
    n_prompt, steps, max_seq = (150, 8, 256) if not wide else (70, 3, 128)
    orc, gpu = make_pair(shape, SEED + 19, 2, max_seq, 8, start_id=1, kv_fill=fill, page_size=ps,
                         n_pages=1 + L * (2 * max_seq // ps))
    gpu.poison_kv()
    orc.poison_kv()
    for slot, n in ((0, n_prompt), (1, 9)):        # the second sequence interleaves its pages
        p = I.prompt_tokens(shape, SEED + 19, slot, n).numpy()
        o = orc.prefill(slot, p)
        g = gpu.d3_prefill(slot, p)
        check_step(f"prefill {slot}", g.cpu().numpy()[None], None, o[None], None)
    toks = I.token_ids(SEED + 19, 5, 64, shape.vocab).numpy()
    for i in range(1, steps + 1):
        for slot in (0, 1):
            r = orc.decode_step([slot], [int(toks[i])], [i], 0.9)
            g, st = gpu.d3_decode_step([slot], [int(toks[i])], [i], 0.9, want_stats=True)
            assert st["kernel_launches"] <= 2, st["kernel_launches"]     # the step, and at most one table patch
            check_step(f"step {i} slot {slot}", g.cpu().numpy(), gpu.d3_read_hidden(1), r["logits"], r["hidden"])
    # cache contents of the first sequence, wherever the oracle's entry is defined
    for l in range(L):
        for t in sorted({min(t, n_prompt + steps - 1) for t in (0, ps - 1, ps, n_prompt - 1, n_prompt, n_prompt + steps - 1)}):
            ok, ov = orc.read_kv(l, 0, t)
            gk, gv = gpu.d3_read_kv(l, 0, t)
            m = np.isfinite(ok)
            assert np.abs(gk[m] - ok[m]).max(initial=0) < 4e-2 and np.abs(gv[m] - ov[m]).max(initial=0) < 4e-2
    gpu.d3_sync()
    gpu.close()


def test_paged_pool_exhaustion_is_an_error_and_changes_nothing(B):
    shape = I.TINY
    L = shape.n_layers
    orc, gpu = make_pair(shape, SEED + 10, 2, 64, 4, page_size=16, n_pages=1 + 2 * L)
    p = I.prompt_tokens(shape, SEED + 10, 0, 16).numpy()
    gpu.d3_prefill(0, p)                       # L pages
    gpu.d3_prefill(1, p[:3])                   # L pages: the pool is now empty
    orc.prefill(0, p)
    assert gpu.d3_kv_pages_used() == 2 * L
    with pytest.raises(B.D3Error) as e:     # position 16 of slot 0 needs a new page per block
        gpu.d3_decode_step([0], [5], [1], 1.0)
    assert e.value.code == B.ECAPACITY
    assert gpu.d3_slot_pos(0) == 16 and gpu.d3_kv_pages_used() == 2 * L
    gpu.d3_reset_slot(1)                       # pages come back; the step now goes through
    r = orc.decode_step([0], [5], [1], 1.0)
    g = gpu.d3_decode_step([0], [5], [1], 1.0)
    check_step("after reset", g.cpu().numpy(), gpu.d3_read_hidden(1), r["logits"], r["hidden"])
    gpu.d3_sync()
    gpu.close()


def test_single_row_call_with_the_least_marshalling(B):
    # the greedy loop's entry of the binding: same C call, one row, against the oracle
    shape = I.TINY
    orc, gpu = make_pair(shape, SEED + 23, 2, 40, 2, start_id=1)
    p = I.prompt_tokens(shape, SEED + 23, 0, 13).numpy()
    tok = O.argmax(orc.prefill(1, p))
    gpu.d3_prefill(1, p)
    lg = torch.empty((1, shape.vocab), dtype=torch.float32, device="cuda:0")
    for i in range(1, 6):
        r = orc.decode_step([1], [tok], [i], 0.9)
        gpu.d3_decode_one(1, tok, i, 0.9, lg)
        check_step(f"step {i}", lg.cpu().numpy(), gpu.d3_read_hidden(1), r["logits"], r["hidden"])
        tok = O.argmax(r["logits"][0])
    with pytest.raises(B.D3Error):
        gpu.d3_decode_one(0, tok, 1, 0.9, lg)      # slot 0 was never prefilled
    gpu.d3_sync()
    gpu.close()


# ------------------------------------------------------------------ error paths

def test_error_paths_change_no_state(B):
    shape = I.TINY
    orc, gpu = make_pair(shape, SEED, 2, 8, 2)
    lg = torch.empty((2, shape.vocab), dtype=torch.float32, device="cuda:0")

    def code(**kw):
        args = dict(slots=[0], tokens=[1], gen_index=[1], alpha=0.9)
        args.update(kw)
        with pytest.raises(B.D3Error) as e:
            gpu.d3_decode_step(**args)
        return e.value.code

    assert code() == B.ESTATE                                   # never prefilled
    gpu.d3_prefill(0, [1, 2, 3])
    gpu.d3_prefill(1, [1, 2, 3])
    assert code(slots=[0, 0], tokens=[1, 1], gen_index=[1, 1]) == B.ESTATE
    assert code(gen_index=[0]) == B.EINVAL
    assert code(tokens=[shape.vocab]) == B.EINVAL
    assert code(slots=[2]) == B.EINVAL
    assert code(alpha=0.0) == B.EINVAL and code(alpha=float("nan")) == B.EINVAL
    assert code(slots=[0, 1, 0], tokens=[1] * 3, gen_index=[1] * 3) == B.ECAPACITY   # > max_batch
    assert gpu.d3_slot_pos(0) == 3 and gpu.d3_slot_pos(1) == 3
    for i in range(5):
        gpu.d3_decode_step([0], [1], [i + 1], 0.9)
    assert code(gen_index=[6]) == B.ECAPACITY                   # cache full
    with pytest.raises(B.D3Error) as e:
        gpu.d3_prefill(1, list(range(9)))
    assert e.value.code == B.ECAPACITY
    gpu.d3_sync()
    gpu.d3_reset_slot(0)
    assert gpu.d3_slot_pos(0) == B.ESTATE
    gpu.close()


def test_argmax_lowest_index_on_ties(B):
    shape = I.TINY
    orc, gpu = make_pair(shape, SEED, 1, 8, 4)
    lg = torch.zeros((4, shape.vocab), dtype=torch.float32, device="cuda:0")
    lg[0, 100] = 3.0
    lg[0, 900] = 3.0
    lg[1, 1023] = 1.0
    lg[2] = -5.0
    lg[3, 0] = 9.0
    out = gpu.d3_argmax(lg).cpu().tolist()
    assert out == [100, 1023, 0, 0]
    gpu.close()
    # a vocabulary that is not a multiple of four (scalar loads) and a large one, random ties
    for vocab in (1003, 32000):
        narrow = I.ModelShape("narrow", 1, 64, 2, 1, 32, 64, vocab)
        orc, gpu = make_pair(narrow, SEED, 1, 8, 4)
        g = torch.Generator().manual_seed(vocab)
        lg = torch.randint(0, 50, (4, vocab), generator=g).float()
        want = [int(np.flatnonzero(r == r.max())[0]) for r in lg.numpy()]
        assert gpu.d3_argmax(lg.to("cuda:0")).cpu().tolist() == want
        gpu.close()
