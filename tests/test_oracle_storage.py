"""Pins of the oracle's bf16 cache-storage rounding (`round_bf16`, used when the oracle is asked to
store K and V in the cache format of the GPU path), and of the size of the effect that this storage
has on the logits.  CPU only."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2503_08524_b200 import inputs as I


def bf16_bits(values) -> np.ndarray:
    """uint16 patterns of doubles that are exactly representable in bf16."""
    f = torch.tensor(np.asarray(values, np.float64)).to(torch.float32)
    assert (f.double().numpy() == np.asarray(values, np.float64)).all() or np.isnan(values).any()
    return (f.view(torch.int32).numpy().astype(np.int64) >> 16) & 0xFFFF


# (input as an exact double, expected bf16 pattern); bf16 = sign, 8 exponent bits, 7 fraction bits
HAND_LISTED = [
    (1.0, 0x3F80),
    (1.0 + 2.0 ** -8, 0x3F80),                # tie between fraction 0 (even) and 1: down
    (1.0 + 3 * 2.0 ** -8, 0x3F82),            # tie between fraction 1 and 2 (even): up
    (1.0 + 2.0 ** -8 + 2.0 ** -30, 0x3F81),   # just above the tie (rounding through fp32 first gives 0x3F80)
    (1.0 + 2.0 ** -8 - 2.0 ** -30, 0x3F80),   # just below the tie
    (1.0 + 3 * 2.0 ** -8 - 2.0 ** -40, 0x3F81),
    (2.0 - 2.0 ** -9, 0x4000),                # carry into the exponent
    (2.0 - 2.0 ** -8, 0x4000),                # tie between 0x3FFF (odd) and 0x4000 (even)
    (2.0 - 3 * 2.0 ** -9, 0x3FFF),
    (-(1.0 + 3 * 2.0 ** -8), 0xBF82),
    (-(1.0 + 2.0 ** -8), 0xBF80),
    (0.0, 0x0000),
    (-0.0, 0x8000),
    (2.0 ** -126, 0x0080),                    # smallest normal
    (2.0 ** -127, 0x0040),                    # subnormal
    (2.0 ** -133, 0x0001),                    # smallest subnormal
    (2.0 ** -134, 0x0000),                    # tie between 0 (even) and the smallest subnormal
    (1.5 * 2.0 ** -134, 0x0001),
    (3 * 2.0 ** -134, 0x0002),                # tie between 1 and 2 (even)
    (-(2.0 ** -135), 0x8000),
    ((2.0 - 2.0 ** -7) * 2.0 ** 127, 0x7F7F),  # largest finite
    ((2.0 - 2.0 ** -8) * 2.0 ** 127, 0x7F80),  # tie above it: the even neighbour is 2^128 = infinity
    ((2.0 - 2.0 ** -8 - 2.0 ** -20) * 2.0 ** 127, 0x7F7F),
    (float("inf"), 0x7F80),
    (float("-inf"), 0xFF80),
]


@pytest.mark.parametrize("real", ["f64", "f32"])
def test_round_bf16_hand_listed_patterns(real):
    xs = np.array([x for x, _ in HAND_LISTED], np.float64)
    want = np.array([b for _, b in HAND_LISTED], np.int64)
    if real == "f32":   # inputs that fp32 cannot hold exactly are not inputs of the fp32 build
        keep = xs.astype(np.float32).astype(np.float64) == xs
        xs, want = xs[keep], want[keep]
    got = O.round_bf16(xs, real=real)
    assert (bf16_bits(got) == want).all(), [(x, hex(g), hex(w)) for x, g, w in zip(xs, bf16_bits(got), want)
                                           if g != w]
    assert (np.signbit(got) == np.signbit(xs)).all()
    assert np.isnan(O.round_bf16(np.array([float("nan")]), real=real))[0]


@pytest.mark.parametrize("real", ["f64", "f32"])
def test_round_bf16_sweep_against_library_conversion(real):
    # every upper half-word (sign, exponent, 7 fraction bits) with 16 different lower halves: ties,
    # near-ties and random bits; fp32 inputs are exact doubles, so one rounding is all there is
    hi = np.arange(65536, dtype=np.int64)
    lows = [0x0000, 0x0001, 0x7FFF, 0x8000, 0x8001, 0xFFFF] + \
        [int(v) for v in I.uniform_ints(11, 3, 10, 0, 0xFFFF)]
    for low in lows:
        bits = ((hi << 16) | low).astype(np.uint32).view(np.int32)
        x = torch.from_numpy(bits.copy()).view(torch.float32)
        finite = torch.isfinite(x)
        want = x.to(torch.bfloat16).double().numpy()
        got = O.round_bf16(x.double().numpy(), real=real)
        f = finite.numpy()
        assert (got[f] == want[f]).all(), low
        assert (np.signbit(got[f]) == np.signbit(want[f])).all(), low


def test_round_bf16_is_idempotent_and_monotone():
    x = np.sort(I.normal_bf16(5, 9, (4096,), "cpu", 1.0).double().numpy() *
                np.linspace(1e-3, 1e3, 4096))
    r = O.round_bf16(x)
    assert (O.round_bf16(r) == r).all()
    assert (np.diff(r) >= 0).all()
    assert (np.abs(r - x) <= np.abs(x) * 2.0 ** -8).all()   # half a unit in the last of 8 bits


def _run_both(shape, seed, P, steps):
    w = I.make_weights(shape, seed, device="cpu", gain_jitter=0.1)
    exact = O.Oracle(shape, w, 1, P + steps + 2, kv_round_bf16=False)
    stored = O.Oracle(shape, w, 1, P + steps + 2, kv_round_bf16=True)
    p = I.prompt_tokens(shape, seed, 0, P).numpy()
    la, lb = exact.prefill(0, p), stored.prefill(0, p)
    diffs, scale = [np.abs(la - lb).max()], np.abs(la).max()
    tok = O.argmax(la)
    for i in range(1, steps + 1):
        ra = exact.decode_step([0], [tok], [i], 1.0)
        rb = stored.decode_step([0], [tok], [i], 1.0)
        diffs.append(np.abs(ra["logits"] - rb["logits"]).max())
        tok = O.argmax(ra["logits"])
    # what the two oracles cached differs by the storage rounding and nothing else
    k0, v0 = exact.read_kv(0, 0, 0)
    k1, v1 = stored.read_kv(0, 0, 0)
    assert (O.round_bf16(k0) == k1).all() and (O.round_bf16(v0) == v1).all()
    return max(diffs), scale


def test_bf16_cache_storage_moves_logits_beyond_the_tolerance_at_7b_width():
    """Why the parity runs at production widths make the oracle store K and V as the cache format
    does: the storage rounding alone (same oracle, same weights, exact against bf16-stored cache)
    moves the largest of the 32000 logits of a 7B-width model by more than the 2e-2 logits tolerance,
    while at the tiny width it stays an order of magnitude below it."""
    small, _ = _run_both(I.TINY, 7, 24, 4)
    assert 1e-4 < small < 5e-3, small
    wide, scale = _run_both(I.LLAMA_7B.with_layers(2), 7, 12, 3)
    assert 2e-2 < wide < 6e-2, wide
    assert wide < 0.02 * scale       # still a small relative effect (logits of magnitude ~5)
