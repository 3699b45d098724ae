"""GPU parity of Eq. 2 with its rotary factors (rotation after the ReLU, numerator only) against the oracle."""
import numpy as np
import pytest

import synth
from parity_util import assert_parity_bf16, assert_parity_f32, to_dev, to_f64

pytestmark = pytest.mark.gpu

EPS = 1e-6


@pytest.fixture(scope="module")
def la():
    import torch

    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2509_24695_b200 as la

    la.load_library()
    return la


def gen(B, N, H, d, seed, dtype):
    return tuple(synth.gauss((B, N, H, d), seed, t, dtype=dtype) for t in (1, 2, 3))


SHAPES = [
    # B, (T, Hh, Ww), H, d
    (1, (3, 8, 8), 4, 32),
    (2, (5, 10, 20), 3, 112),    # several tiles and a ragged tail at the paper's head dim
    (1, (1, 1, 129), 2, 112),
    (1, (1, 1, 1), 1, 112),
    (1, (2, 7, 11), 2, 128),
    (2, (4, 9, 20), 5, 128),     # tensor-core path at d = 128: several tiles, trailing CTAs, a ragged tail
    (2, (3, 5, 7), 5, 64),
    (2, (4, 9, 20), 5, 64),      # packed heads on the tensor cores: two per operand, an odd head count, a ragged tail
    (1, (5, 10, 20), 7, 32),     # four per operand, the last group with three heads
    (2, (2, 7, 11), 9, 32),
    (1, (2, 5, 9), 3, 6),
]


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "B%d_T%dx%dx%d_H%d_d%d" % (s[0], *s[1], s[2], s[3]))
def test_rope_forward_matches_oracle(la, orc, shape, dtype):
    B, (T, Hh, Ww), H, d = shape
    N = T * Hh * Ww
    q, k, v = gen(B, N, H, d, 5000 + N + d, dtype)
    cos, sin = synth.rope_table(T, Hh, Ww, d)
    table = la.rope_pack(to_dev(cos), to_dev(sin))
    # the operation is defined on the packed fp16 (cos, sin) values: the oracle gets exactly those
    packed = table.cpu().numpy().astype(np.float64)
    assert np.array_equal(packed[..., 0], cos.astype(np.float16).astype(np.float64))
    assert np.array_equal(packed[..., 1], sin.astype(np.float16).astype(np.float64))
    ref = orc.rope_forward(q, k, v, packed[..., 0], packed[..., 1], EPS)
    o = la.linattn_forward_rope(to_dev(q), to_dev(k), to_dev(v), table, EPS)
    (assert_parity_bf16 if dtype == "bf16" else assert_parity_f32)(to_f64(o), ref, f"rope forward {shape} {dtype}")


def test_rope_with_zero_angles_is_the_plain_forward(la):
    import torch

    q, k, v = (to_dev(x) for x in gen(1, 700, 3, 112, 5100, "bf16"))
    one = torch.ones((700, 56), dtype=torch.float32, device="cuda")
    o = la.linattn_forward_rope(q, k, v, la.rope_pack(one, torch.zeros_like(one)), EPS)
    ref = la.linattn_forward(q, k, v, EPS)
    # same mathematics; the two run different kernels, so compare within output rounding
    assert_parity_bf16(to_f64(o), to_f64(ref), "zero angles")


def test_rope_errors(la):
    import torch

    x = torch.zeros((1, 8, 2, 7), dtype=torch.bfloat16, device="cuda")
    t = torch.zeros((8, 3, 2), dtype=torch.float16, device="cuda")
    with pytest.raises(la.LinAttnError) as e:
        la.linattn_forward_rope(x, x.clone(), x.clone(), t, EPS)
    assert e.value.status == -2   # odd head dim: features cannot be paired


@pytest.mark.parametrize("case", [("bf16", 3, 112, (7, 6, 10), 60), ("f32", 2, 112, (4, 5, 5), 25), ("bf16", 2, 64, (6, 4, 8), 64),
                                  ("bf16", 2, 112, (3, 1, 150), 150), ("bf16", 3, 128, (5, 7, 9), 130), ("bf16", 6, 32, (6, 4, 8), 64),
                                  ("bf16", 3, 64, (5, 7, 9), 130)],
                         ids=lambda c: "%s_H%d_d%d_Tb%d" % (c[0], c[1], c[2], c[4]))
def test_rope_block_steps_match_the_block_causal_oracle(la, orc, case):
    """Cached block-by-block generation with rotary factors against the oracle's block-causal form; the last
    block also equals the tail of the bidirectional rotary forward, and the cache size stays constant."""
    import torch

    dtype, H, d, (T, Hh, Ww), T_b = case
    B, N = 1, T * Hh * Ww
    q, k, v = gen(B, N, H, d, 5200 + N + d, dtype)
    cos, sin = synth.rope_table(T, Hh, Ww, d)
    table = la.rope_pack(to_dev(cos), to_dev(sin))
    packed = table.cpu().numpy().astype(np.float64)
    ref = orc.rope_forward(q, k, v, packed[..., 0], packed[..., 1], EPS, T_b=T_b)
    check = assert_parity_bf16 if dtype == "bf16" else assert_parity_f32
    cache = la.BlockLinCache(B, H, d, torch.bfloat16 if dtype == "bf16" else torch.float32, "cuda", max_T_b=T_b, eps=EPS)
    bytes0 = cache.info()["state_bytes"]
    outs = []
    for n0 in range(0, N, T_b):
        sl = slice(n0, min(n0 + T_b, N))
        blk = [to_dev(np.ascontiguousarray(x[:, sl])) for x in (q, k, v)]
        outs.append(cache.step_rope(*blk, table[sl].contiguous()))
        assert cache.info()["state_bytes"] == bytes0 == B * H * (d * d + d) * 4
    stepped = torch.cat(outs, dim=1)
    check(to_f64(stepped), ref, f"rope steps {case}")
    full = la.linattn_forward_rope(to_dev(q), to_dev(k), to_dev(v), table, EPS)
    last = (N - 1) // T_b * T_b
    check(to_f64(stepped[:, last:]), to_f64(full[:, last:]).copy(), "last block vs bidirectional rotary forward")


def tdtype(dtype):
    import torch

    return torch.bfloat16 if dtype == "bf16" else torch.float32


def packed_table(la, T, Hh, Ww, d):
    cos, sin = synth.rope_table(T, Hh, Ww, d)
    table = la.rope_pack(to_dev(cos), to_dev(sin))
    packed = table.cpu().numpy().astype(np.float64)
    return table, packed[..., 0], packed[..., 1]


@pytest.mark.parametrize("dtype,d", [("bf16", 112), ("f32", 112), ("bf16", 64), ("bf16", 6), ("bf16", 128), ("bf16", 32)])
def test_rope_denoise_loop_reads_without_committing(la, orc, dtype, d):
    """Algorithm 1 on the attention the model runs (Eq. 2 with RoPE): every denoising step of a block reads the
    rotary cache together with the noisy block itself and leaves the cache as it was; only the clean block is
    committed.  The oracle's step runs on a copy of its cache."""
    import torch

    B, H, (T, Hh, Ww), fb, M, steps = 1, 3, (6, 10, 15), 2, 3, 2    # blocks of fb = 2 frames = 300 tokens
    T_b = fb * Hh * Ww
    table, cs, sn = packed_table(la, T, Hh, Ww, d)
    check = assert_parity_bf16 if dtype == "bf16" else assert_parity_f32
    cache = la.BlockLinCache(B, H, d, tdtype(dtype), "cuda", max_T_b=T_b, eps=EPS)
    ocache = orc.new_cache(B, H, d)
    for blk in range(M):
        sl = slice(blk * T_b, (blk + 1) * T_b)
        tab = table[sl].contiguous()
        before = cache.state.clone()
        for j in range(steps):          # noisy versions of the block: other values each time, same positions
            q, k, v = gen(B, T_b, H, d, 5400 + 10 * blk + j, dtype)
            o = cache.peek_rope(to_dev(q), to_dev(k), to_dev(v), tab)
            ref = orc.rope_block_step((ocache[0].copy(), ocache[1].copy()), q, k, v, cs[sl], sn[sl], EPS)
            check(to_f64(o), ref, f"rotary peek block {blk} step {j}")
            assert torch.equal(cache.state, before), "a read-only step changed the cache"
            assert cache.info()["blocks_seen"] == blk
        q, k, v = gen(B, T_b, H, d, 5500 + blk, dtype)               # the clean block
        o_peek = cache.peek_rope(to_dev(q), to_dev(k), to_dev(v), tab)
        o_step = cache.step_rope(to_dev(q), to_dev(k), to_dev(v), tab)
        assert torch.equal(o_peek, o_step)                            # same arithmetic, committed or not
        check(to_f64(o_step), orc.rope_block_step(ocache, q, k, v, cs[sl], sn[sl], EPS), f"rotary step block {blk}")
        S, z = ocache
        got = to_f64(cache.state)
        # z sums the plain features in fp32.  S sums rotated features: fp32 throughout on the fp32 path; on the bf16
        # path the rotated key is rounded to bf16 before it enters the tensor core (2^-9 relative per term, unbiased:
        # the sum's error is about 1.5e-3 of the state's RMS, its largest of 37 632 entries several times that)
        for g, r, name, rel in ((got[..., :d, :].swapaxes(-1, -2), S, "S", 1e-2 if (dtype == "bf16" and d in (32, 64, 112, 128)) else 1e-5),
                                (got[..., d, :], z, "z", 1e-5)):
            rms = np.sqrt((r ** 2).mean(axis=tuple(range(2, r.ndim)), keepdims=True))
            assert (np.abs(g - r) <= rel * (np.abs(r) + rms)).all(), f"rotary cache after block {blk}: {name}"
    assert cache.info()["blocks_seen"] == M and cache.status() == 0


@pytest.mark.parametrize("case", [("bf16", 3, 112, (6, 6, 10), 2), ("f32", 2, 112, (4, 5, 5), 1), ("bf16", 2, 64, (6, 4, 8), 3),
                                  ("bf16", 2, 6, (4, 3, 5), 2), ("bf16", 4, 128, (6, 5, 9), 2), ("bf16", 5, 32, (6, 4, 8), 2)],
                         ids=lambda c: "%s_H%d_d%d_fb%d" % (c[0], c[1], c[2], c[4]))
def test_rope_prefill_equals_steps_and_oracle(la, orc, case):
    """blocklin_prefill_rope over all blocks: the bits of single rotary steps, the oracle's block-causal rotary form,
    and (absorb only: q = o = NULL) the same cache."""
    import torch

    dtype, H, d, (T, Hh, Ww), fb = case
    B, N, T_b = 2, T * Hh * Ww, fb * Hh * Ww
    M = N // T_b
    q, k, v = gen(B, N, H, d, 5600 + N + d, dtype)
    table, cs, sn = packed_table(la, T, Hh, Ww, d)
    qd, kd, vd = to_dev(q), to_dev(k), to_dev(v)
    check = assert_parity_bf16 if dtype == "bf16" else assert_parity_f32
    cache = la.BlockLinCache(B, H, d, tdtype(dtype), "cuda", max_T_b=T_b, eps=EPS, strides=tuple(qd.stride()[:3]))
    stepped = torch.empty_like(qd)       # blocks are token ranges of the long tensors: they keep its batch stride
    for i in range(M):
        sl = slice(i * T_b, (i + 1) * T_b)
        cache.step_rope(qd[:, sl], kd[:, sl], vd[:, sl], table[sl], out=stepped[:, sl])
    final = cache.state.clone()
    cache.reset()
    assert (cache.state == 0).all()
    o = cache.prefill_rope(qd, kd, vd, table, M)
    assert torch.equal(o, stepped) and torch.equal(cache.state, final)
    assert cache.info() == {"blocks_seen": M, "tokens_seen": N, "state_bytes": B * H * (d * d + d) * 4}
    check(to_f64(o), orc.rope_forward(q, k, v, cs, sn, EPS, T_b=T_b), f"rotary prefill {case}")
    cache.reset()
    assert cache.prefill_rope(None, kd, vd, table, M) is None        # context only
    assert torch.equal(cache.state, final) and cache.status() == 0
