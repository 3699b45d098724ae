"""Pins of the temporal-convolution oracle (oracle/tconv.py) against things other than itself: library
routines (numpy's correlate, scipy's lfilter) in the special cases that reduce to them, impulse responses
written out by hand, causality, the identity at zero taps, exact small-integer arithmetic, and the
equality of the one-shot block form with cached stepping.  ``test_mutants_are_caught`` plants plausible
mistakes in a copy of the oracle's source and requires that some pin rejects each."""
import importlib.util
import os

import numpy as np
import pytest

from oracle import tconv as tconv_mod

SOURCE = os.path.abspath(tconv_mod.__file__)


def _x(B, T, HW, D, seed):
    return np.random.default_rng(seed).normal(size=(B, T, HW, D))


def _w(D, seed):
    return np.random.default_rng(seed).normal(size=(3, D))


def pin_bidirectional_is_library_correlation(o):
    """Per (batch, position, channel) the layer is x + correlate(x, w, 'same') along the frames."""
    B, T, HW, D = 2, 7, 3, 4
    x, w = _x(B, T, HW, D, 1), _w(D, 2)
    y = o.tconv_bidirectional(x, w)
    for b in range(B):
        for p in range(HW):
            for c in range(D):
                ref = x[b, :, p, c] + np.correlate(x[b, :, p, c], w[:, c], mode="same")
                np.testing.assert_allclose(y[b, :, p, c], ref, rtol=1e-13, atol=1e-13)


def pin_blocks_of_one_frame_are_a_causal_filter(o):
    """T_b = 1: no next frame is ever seen; y = x + lfilter([w1, w0], [1], x) along the frames."""
    from scipy.signal import lfilter

    B, T, HW, D = 1, 9, 2, 3
    x, w = _x(B, T, HW, D, 3), _w(D, 4)
    y = o.tconv_block_masked(x, w, 1)
    for p in range(HW):
        for c in range(D):
            ref = x[0, :, p, c] + lfilter([w[1, c], w[0, c]], [1.0], x[0, :, p, c])
            np.testing.assert_allclose(y[0, :, p, c], ref, rtol=1e-13, atol=1e-13)


def pin_impulse_responses(o):
    """A unit impulse in one frame, position and channel: the taps land where the definition puts them."""
    B, T, HW, D, T_b = 1, 6, 2, 3, 3
    w = np.array([[2.0, 3.0, 5.0], [7.0, 11.0, 13.0], [17.0, 19.0, 23.0]])   # w[tau][c]
    for t0 in range(T):
        x = np.zeros((B, T, HW, D)); x[0, t0, 1, 2] = 1.0
        want = np.zeros_like(x)
        want[0, t0, 1, 2] = 1.0 + w[1, 2]
        if t0 + 1 < T:
            want[0, t0 + 1, 1, 2] = w[0, 2]            # the next frame sees it as its previous frame
        bi = want.copy()
        if t0 > 0:
            bi[0, t0 - 1, 1, 2] = w[2, 2]              # the frame before sees it as its next frame
        assert np.array_equal(o.tconv_bidirectional(x, w), bi)
        blk = want.copy()
        if t0 > 0 and t0 % T_b != 0:                    # ... unless a block boundary lies between them
            blk[0, t0 - 1, 1, 2] = w[2, 2]
        assert np.array_equal(o.tconv_block_masked(x, w, T_b), blk)


def pin_zero_taps_is_identity_and_centre_tap_scales(o):
    x = _x(2, 5, 3, 4, 5)
    zero = np.zeros((3, 4))
    assert np.array_equal(o.tconv_bidirectional(x, zero), x)
    assert np.array_equal(o.tconv_block_masked(x, zero, 2), x)
    y, f = o.tconv_block_step(x, zero, o.new_cache(2, 3, 4) + 9.0)
    assert np.array_equal(y, x) and np.array_equal(f, x[:, -1])
    centre = np.zeros((3, 4)); centre[1] = [1.0, 2.0, 3.0, -1.0]
    assert np.allclose(o.tconv_bidirectional(x, centre), x * (1.0 + centre[1]), rtol=1e-15)


def pin_causality_across_blocks(o):
    """Frames of later blocks never change earlier blocks' outputs; within a block both neighbours count."""
    B, T, HW, D, T_b = 1, 8, 2, 3, 3
    x, w = _x(B, T, HW, D, 6), _w(D, 7)
    y = o.tconv_block_masked(x, w, T_b)
    x2 = x.copy(); x2[:, 6:] += 1.0
    y2 = o.tconv_block_masked(x2, w, T_b)
    assert np.array_equal(y2[:, :6], y[:, :6]) and not np.array_equal(y2[:, 6:], y[:, 6:])
    x3 = x.copy(); x3[:, 5] += 1.0                       # last frame of block 1
    y3 = o.tconv_block_masked(x3, w, T_b)
    assert np.array_equal(y3[:, :4], y[:, :4])           # block 0 and frame 3 (not a neighbour) untouched
    assert not np.array_equal(y3[:, 4], y[:, 4])         # its own block sees it (as the next frame)
    assert not np.array_equal(y3[:, 6], y[:, 6])         # the next block sees it through the cache
    assert np.array_equal(y3[:, 7], y[:, 7])
    # one block over everything is the bidirectional layer
    assert np.array_equal(o.tconv_block_masked(x, w, T), o.tconv_bidirectional(x, w))


def pin_stepping_equals_one_shot(o):
    for (B, T, HW, D, T_b) in [(2, 9, 3, 4, 3), (1, 8, 2, 5, 3), (1, 4, 1, 2, 1), (1, 5, 2, 2, 5)]:
        x, w = _x(B, T, HW, D, 8 + T), _w(D, 9)
        ref = o.tconv_block_masked(x, w, T_b)
        f = o.new_cache(B, HW, D)
        assert f.size == o.cache_elems(B, HW, D) == B * HW * D
        outs = []
        for t0 in range(0, T, T_b):
            blk = x[:, t0:t0 + T_b]
            peek, f_same = o.tconv_block_step(blk + 0.5, w, f, commit=False)   # a denoising step reads only
            assert f_same is f or np.array_equal(f_same, f)
            y, f = o.tconv_block_step(blk, w, f)
            assert f.size == B * HW * D                  # the cache never grows
            assert np.array_equal(f, blk[:, -1])
            outs.append(y)
        assert np.array_equal(np.concatenate(outs, axis=1), ref)


def pin_bf16_bits_and_small_integers(o):
    """bf16 inputs are widened exactly; with small integers every result is an exact integer."""
    bits = np.array([0x3F80, 0xBF80, 0x4000, 0x0000, 0x4040, 0xC080], dtype=np.uint16)   # 1 -1 2 0 3 -4
    assert np.array_equal(o.widen(bits), [1.0, -1.0, 2.0, 0.0, 3.0, -4.0])
    x = bits.reshape(1, 3, 1, 2)                          # frames: (1,-1) (2,0) (3,-4)
    w = np.array([[1.0, 2.0], [10.0, 20.0], [100.0, 200.0]])
    y = o.tconv_bidirectional(x, w)
    # channel 0: x = 1 2 3 ; channel 1: x = -1 0 -4
    assert np.array_equal(y[0, :, 0, 0], [1 + 10 + 200, 2 + 1 + 20 + 300, 3 + 2 + 30])
    assert np.array_equal(y[0, :, 0, 1], [-1 - 20 + 0, 0 - 2 + 0 - 800, -4 + 0 - 80])


def pin_golden_hand_worked(o):
    """tests/golden/tconv_hand_worked.txt: four frames, two channels, worked by hand (derivation in the file)."""
    import sys

    sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
    from parity_util import read_golden

    g = read_golden("tconv_hand_worked.txt")
    x = g["x"].reshape(1, 4, 1, 2)
    assert np.array_equal(o.tconv_bidirectional(x, g["w"])[0, :, 0], g["y_bidirectional"])
    assert np.array_equal(o.tconv_block_masked(x, g["w"], 2)[0, :, 0], g["y_blocks_of_two"])
    f = o.new_cache(1, 1, 2)
    ys = []
    for t0 in (0, 2):
        y, f = o.tconv_block_step(x[:, t0:t0 + 2], g["w"], f)
        ys.append(y)
    assert np.array_equal(np.concatenate(ys, axis=1)[0, :, 0], g["y_blocks_of_two"])
    assert np.array_equal(f[0, 0], g["cache_after"][0])


PINS = [pin_golden_hand_worked, pin_bidirectional_is_library_correlation, pin_blocks_of_one_frame_are_a_causal_filter, pin_impulse_responses,
        pin_zero_taps_is_identity_and_centre_tap_scales, pin_causality_across_blocks, pin_stepping_equals_one_shot,
        pin_bf16_bits_and_small_integers]


@pytest.mark.parametrize("pin", PINS, ids=lambda f: f.__name__)
def test_pin(pin):
    pin(tconv_mod)


MUTANTS = {
    "taps_reversed": ("return cur + w[0] * prev + w[1] * cur + w[2] * nxt", "return cur + w[2] * prev + w[1] * cur + w[0] * nxt"),
    "shortcut_dropped": ("return cur + w[0] * prev", "return w[0] * prev"),
    "centre_tap_dropped": ("+ w[1] * cur ", "+ 0 * cur "),
    "taps_shared_over_channels": ("return cur + w[0] * prev + w[1] * cur + w[2] * nxt",
                                  "return cur + w[0][0] * prev + w[1][0] * cur + w[2][0] * nxt"),
    "block_sees_next_block": ("        nxt = zero if last_of_block else x[:, t + 1]\n",
                              "        nxt = zero if t + 1 == T else x[:, t + 1]\n"),
    "block_forgets_previous_block": ("        prev = x[:, t - 1] if t > 0 else zero                    # same block",
                                     "        prev = x[:, t - 1] if t % T_b else zero                    # same block"),
    "boundary_off_by_one": ("last_of_block = (t + 1) % T_b == 0 or t + 1 == T", "last_of_block = t % T_b == 0 or t + 1 == T"),
    "cache_keeps_first_frame": ("new = x[:, T - 1].copy()", "new = x[:, 0].copy()"),
    "cache_not_replaced": ("new = x[:, T - 1].copy() if (commit and T > 0) else cache", "new = cache"),
    "peek_commits": ("if (commit and T > 0) else cache", "if T > 0 else cache"),
    "step_without_zero_frame": ("padded = np.concatenate([cache[:, None], x, np.zeros((B, 1, HW, D))], axis=1)",
                                "padded = np.concatenate([cache[:, None], x, x[:, -1:]], axis=1)"),
    "step_ignores_cache": ("padded = np.concatenate([cache[:, None], x,", "padded = np.concatenate([0 * cache[:, None], x,"),
    "bidirectional_wraps_around": ("        prev = x[:, t - 1] if t > 0 else zero\n        nxt = x[:, t + 1] if t + 1 < T else zero\n",
                                   "        prev = x[:, t - 1]\n        nxt = x[:, (t + 1) % T]\n"),
    "bf16_shift": ("<< 16)", "<< 15)"),
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_mutants_are_caught(tmp_path, name):
    old, new = MUTANTS[name]
    src = open(SOURCE).read()
    assert src.count(old) >= 1, f"mutation site for {name} not found in the oracle source"
    p = tmp_path / f"tconv_mutant_{name}.py"
    p.write_text(src.replace(old, new))
    spec = importlib.util.spec_from_file_location(f"tconv_mutant_{name}", str(p))
    mutant = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mutant)
    caught = []
    for pin in PINS:
        try:
            with np.errstate(all="ignore"):
                pin(mutant)
        except (AssertionError, IndexError, ValueError):
            caught.append(pin.__name__)
    assert caught, f"no pin rejects the planted mistake '{name}'"
