"""GPU parity of the temporal convolution of the Mix-FFN (tconv.h) against the fp64 oracle (oracle/tconv.py).

Tolerance.  Per output element the kernel does three fp32 fused multiply-adds on exactly widened inputs and
(bf16) one rounding to nearest even at the store.  With mag = |x| + |w0 x_prev| + |w1 x| + |w2 x_next| the fp32
part is within 3 * 2^-24 * mag of the exact value, and the bf16 rounding adds at most 2^-8 * |y| (bf16 keeps 8 significant bits):
  bf16:  |delta| <= 2^-8 * |ref| + 4 * 2^-24 * mag        fp32:  |delta| <= 4 * 2^-24 * mag
Small-integer inputs must come out bit for bit.
"""
import numpy as np
import pytest

from oracle import tconv as orc_conv
import synth
from parity_util import to_dev, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def la():
    import torch

    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2509_24695_b200 as la

    la.load_library()
    return la


def tdtype(dtype):
    import torch

    return torch.bfloat16 if dtype == "bf16" else torch.float32


def magnitude(x, w, T_b=None, cache=None):
    """|x| + sum of |tap * neighbour| in the block-causal (or bidirectional, T_b None) neighbourhood."""
    ax = np.abs(orc_conv.widen(x))
    aw = np.abs(np.asarray(w, dtype=np.float64))
    if T_b is None:
        return orc_conv.tconv_bidirectional(ax, aw)
    if cache is None:
        return orc_conv.tconv_block_masked(ax, aw, T_b)
    return orc_conv.tconv_block_step(ax, aw, np.abs(cache), commit=False)[0]


def check(got, ref, mag, dtype, what):
    assert got.shape == ref.shape and np.isfinite(got).all(), what
    bound = 4 * 2.0 ** -24 * mag + (2.0 ** -8 * np.abs(ref) if dtype == "bf16" else 0.0)
    delta = np.abs(got - ref)
    assert (delta <= bound).all(), f"{what}: worst ratio {(delta / (bound + 1e-300)).max():.3f}"


def gen(B, T, HW, D, seed, dtype):
    w = synth.ConvWorkload("case", B=B, T=T, HW=HW, D=D, seed=seed)
    return synth.conv_frames(w, dtype), synth.conv_taps(D, seed)


# (B, T, HW, D, T_b): one and several thread blocks per frame, ragged tails, blocks of 1 frame, one big block
CASES = [
    (2, 5, 6, 16, 2),
    (1, 7, 37, 72, 3),      # 333 16-byte columns: two thread blocks, the second ragged
    (2, 6, 130, 40, 3),
    (1, 4, 9, 2240, 1),     # the model width
    (3, 3, 5, 8, 3),
    (1, 1, 11, 24, 1),      # a single frame
    (1, 3, 9, 16, 1),       # three one-frame blocks in one prefill: every block ends with the zero frame
    (2, 2, 9, 16, 1),       # two one-frame blocks, two batch entries
    (1, 3, 130, 40, 3),     # one three-frame block: the short-step kernel
]


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("case", CASES, ids=lambda c: "B%d_T%d_HW%d_D%d_Tb%d" % c)
def test_forward_steps_and_prefill(la, case, dtype):
    import torch

    B, T, HW, D, T_b = case
    x, w = gen(B, T, HW, D, 4000 + HW + D, dtype)
    xd, wd = to_dev(x), to_dev(w)
    launches0 = la.kernel_launches()

    # bidirectional layer (Sec. 3.1)
    y = la.tconv_forward(xd, wd)
    assert la.kernel_launches() == launches0 + 1
    check(to_f64(y), orc_conv.tconv_bidirectional(x, w), magnitude(x, w), dtype, f"forward {case}")

    # block-causal: cached steps against the one-shot block form (Sec. 3.2)
    ref = orc_conv.tconv_block_masked(x, w, T_b)
    mag = magnitude(x, w, T_b)
    cache = la.TConvCache(B, HW, D, tdtype(dtype), "cuda")
    assert cache.frame.numel() == B * HW * D and (cache.frame == 0).all()
    outs = []
    f = orc_conv.new_cache(B, HW, D)
    for t0 in range(0, T, T_b):
        blk = xd[:, t0:t0 + T_b]                       # a sub-view of the long tensor: batch stride T*HW*D
        before = cache.frame.clone()
        peek = cache.step(blk, wd, commit=False)        # a denoising step of Algorithm 1 reads the cache only
        assert torch.equal(cache.frame, before)
        yb = cache.step(blk, wd)
        assert torch.equal(peek, yb)
        assert torch.equal(cache.frame, xd[:, min(t0 + T_b, T) - 1])   # the cache is the block's last frame ...
        assert cache.frame.numel() == B * HW * D                       # ... and nothing else, at every step
        y_o, f = orc_conv.tconv_block_step(x[:, t0:t0 + T_b], w, f)
        check(to_f64(yb), y_o, mag[:, t0:t0 + T_b], dtype, f"step at frame {t0} {case}")
        outs.append(yb)
    stepped = torch.cat(outs, dim=1)
    check(to_f64(stepped), ref, mag, dtype, f"steps vs one-shot block form {case}")

    # all blocks in one launch: the same bits and the same cache
    if T % T_b == 0:
        final = cache.frame.clone()
        cache.reset()
        assert (cache.frame == 0).all()
        launches0 = la.kernel_launches()
        y_all = cache.prefill(xd, wd, T // T_b)
        assert la.kernel_launches() == launches0 + 1
        assert torch.equal(y_all, stepped) and torch.equal(cache.frame, final)
        # and it continues from a non-empty cache
        y_again = cache.prefill(xd, wd, T // T_b)
        y_o, _ = orc_conv.tconv_block_step(x[:, :T_b], w, orc_conv.widen(x[:, -1]))
        check(to_f64(y_again[:, :T_b]), y_o, magnitude(x[:, :T_b], w, T_b, orc_conv.widen(x[:, -1])), dtype,
              "first block after a full pass")
        assert torch.equal(y_again[:, T_b:], stepped[:, T_b:])

    # absorb without output
    cache.reset()
    cache.absorb(xd[:, :T_b])
    assert torch.equal(cache.frame, xd[:, min(T_b, T) - 1])


def test_small_integers_are_exact(la):
    import torch

    B, T, HW, D, T_b = 2, 9, 50, 64, 3
    x = synth.smallint((B, T, HW, D), 4100, synth.X_ID, 2)
    w = synth.smallint((3, D), 4101, synth.W_ID, 2)
    wf = orc_conv.widen(w).astype(np.float32)
    xd, wd = to_dev(x), to_dev(wf)
    assert np.array_equal(to_f64(la.tconv_forward(xd, wd)), orc_conv.tconv_bidirectional(x, wf))
    cache = la.TConvCache(B, HW, D, torch.bfloat16, "cuda")
    assert np.array_equal(to_f64(cache.prefill(xd, wd, T // T_b)), orc_conv.tconv_block_masked(x, wf, T_b))


def test_zero_taps_is_identity(la):
    """The shortcut alone: with all taps zero the layer returns its input, bit for bit."""
    import torch

    x, _ = gen(1, 4, 33, 48, 4200, "bf16")
    xd = to_dev(x)
    assert torch.equal(la.tconv_forward(xd, torch.zeros(3, 48, device="cuda")), xd)


def test_errors_and_empty(la):
    import torch

    w = torch.zeros(3, 16, device="cuda")
    x = torch.zeros(1, 2, 4, 16, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(la.LinAttnError) as e:      # y must not be x
        la.tconv_forward(x, w, out=x)
    assert e.value.status == -1
    x12 = torch.zeros(1, 2, 4, 12, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(la.LinAttnError) as e:      # channels not a multiple of 8
        la.tconv_forward(x12, torch.zeros(3, 12, device="cuda"))
    assert e.value.status == -2
    with pytest.raises(ValueError):
        la.tconv_forward(x, torch.zeros(3, 8, device="cuda"))
    cache = la.TConvCache(1, 4, 16, torch.bfloat16, "cuda")
    with pytest.raises(ValueError):
        cache.step(torch.zeros(1, 2, 5, 16, dtype=torch.bfloat16, device="cuda"), w)
    # zero frames: a successful no-op
    n0 = la.kernel_launches()
    empty = torch.zeros(1, 0, 4, 16, dtype=torch.bfloat16, device="cuda")
    assert la.tconv_forward(empty, w).shape == (1, 0, 4, 16)
    cache.step(empty, w)
    assert la.kernel_launches() == n0 and (cache.frame == 0).all()


def _sampled_positions(HW, count, seed):
    rng = np.random.default_rng(seed)
    return np.unique(np.concatenate([[0, 1, HW // 2, HW - 2, HW - 1], rng.integers(0, HW, size=count)]))


@pytest.mark.parametrize("wl", [synth.CONV_P480, synth.CONV_P720], ids=lambda w: w.name)
def test_full_size_bidirectional(la, wl):
    """The 480p / 720p layers in the launch configuration the benchmark times; every frame and channel of
    sampled positions against the oracle (positions and channels are independent of one another)."""
    import torch

    x = synth.conv_frames(wl)
    w = synth.conv_taps(wl.D, wl.seed)
    y = la.tconv_forward(to_dev(x), to_dev(w))
    pos = _sampled_positions(wl.HW, 40, wl.seed)
    xs = np.ascontiguousarray(x[:, :, pos])
    check(to_f64(y[:, :, torch.from_numpy(pos).cuda()]), orc_conv.tconv_bidirectional(xs, w), magnitude(xs, w), "bf16", wl.name)
    assert torch.isfinite(y.float()).all()


@pytest.mark.parametrize("wl", [synth.CONV_AR480, synth.CONV_STREAM720], ids=lambda w: w.name)
def test_full_size_block_causal(la, wl):
    """Blocks of 3 frames at the 480p / 720p sizes, stepped with the cache; sampled positions against the
    one-shot block form; the cache stays one frame."""
    import torch

    x = synth.conv_frames(wl)
    w = synth.conv_taps(wl.D, wl.seed)
    xd, wd = to_dev(x), to_dev(w)
    cache = la.TConvCache(wl.B, wl.HW, wl.D, torch.bfloat16, "cuda")
    outs = []
    for t0 in range(0, wl.T, wl.T_b):
        outs.append(cache.step(xd[:, t0:t0 + wl.T_b], wd))
        assert cache.frame.numel() * 2 == wl.B * wl.HW * wl.D * 2
    y = torch.cat(outs, dim=1)
    pos = _sampled_positions(wl.HW, 24, wl.seed)
    xs = np.ascontiguousarray(x[:, :, pos])
    check(to_f64(y[:, :, torch.from_numpy(pos).cuda()]), orc_conv.tconv_block_masked(xs, w, wl.T_b),
          magnitude(xs, w, wl.T_b), "bf16", wl.name)
    assert torch.equal(cache.frame, xd[:, -1])
    cache.reset()
    assert torch.equal(cache.prefill(xd, wd, wl.T // wl.T_b), y)


def test_hand_worked_example_on_the_gpu(la):
    """The hand-worked example of tests/golden/tconv_hand_worked.txt through the library (fp32 path; its two channels
    repeated to the four the 16-byte pieces need, at three positions)."""
    import torch
    from parity_util import read_golden

    g = read_golden("tconv_hand_worked.txt")
    tile = lambda a: np.tile(a, (1, 2)).astype(np.float32)            # [T or 3, 2] -> [.., 4]
    x = torch.from_numpy(np.repeat(tile(g["x"])[None, :, None, :], 3, axis=2)).cuda().contiguous()   # [1, 4, 3, 4]
    w = torch.from_numpy(tile(g["w"])).cuda().contiguous()
    y = to_f64(la.tconv_forward(x, w))
    assert all(np.array_equal(y[0, :, p], tile(g["y_bidirectional"])) for p in range(3))
    cache = la.TConvCache(1, 3, 4, torch.float32, "cuda")
    yb = to_f64(torch.cat([cache.step(x[:, t0:t0 + 2], w) for t0 in (0, 2)], dim=1))
    assert all(np.array_equal(yb[0, :, p], tile(g["y_blocks_of_two"])) for p in range(3))
    assert np.array_equal(to_f64(cache.frame)[0, 0], tile(g["cache_after"])[0])
