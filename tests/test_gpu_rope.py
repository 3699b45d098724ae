"""GPU parity of Eq. 2 with its rotary factors (rotation after the ReLU, numerator only) against the oracle."""
import numpy as np
import pytest

from paper_2509_24695_b200 import synth
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
    (2, (3, 5, 7), 5, 64),
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
                                  ("bf16", 2, 112, (3, 1, 150), 150)],
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
