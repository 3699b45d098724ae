"""GPU parity: the CUDA path (through the C ABI) against the fp64 CPU oracle, element by element,
on the same seeded inputs.  Sizes here span several tiles and ragged tails but stay small enough
for the oracle to finish in seconds; the full-size workloads are in test_gpu_fullsize.py."""
import numpy as np
import pytest

import synth
from parity_util import assert_parity_bf16, assert_parity_f32, assert_state_close, to_dev, to_f64

pytestmark = pytest.mark.gpu

EPS = 1e-6


@pytest.fixture(scope="module")
def la():
    import torch

    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2509_24695_b200 as la

    la.load_library()
    return la


def gen(B, N, H, d, seed, dtype, scale=1.0):
    return tuple(synth.gauss((B, N, H, d), seed, t, scale=scale, dtype=dtype) for t in (1, 2, 3))


def check(dtype, got, ref, what):
    (assert_parity_bf16 if dtype == "bf16" else assert_parity_f32)(got, ref, what)


SHAPES = [
    # B, N, H, d
    (1, 192, 4, 32),      # config 1
    (2, 1000, 3, 112),    # several 128-token tiles + ragged tail, the paper's head dim
    (1, 129, 2, 112),
    (1, 127, 2, 112),
    (1, 1, 1, 112),
    (1, 2, 5, 64),
    (2, 777, 5, 64),
    (1, 515, 7, 32),      # head count not a multiple of the 4-head packing
    (2, 300, 3, 128),
    (1, 333, 2, 16),      # head dims outside the tensor-core set
    (1, 77, 3, 7),
    (1, 260, 1, 96),
]


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "B%d_N%d_H%d_d%d" % s)
def test_forward_matches_oracle(la, orc, shape, dtype):
    B, N, H, d = shape
    q, k, v = gen(B, N, H, d, 2000 + N + d, dtype)
    ref = orc.forward(q, k, v, EPS)
    o = la.linattn_forward(to_dev(q), to_dev(k), to_dev(v), EPS)
    check(dtype, to_f64(o), ref, f"forward {shape} {dtype}")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("shape", [(2, 1000, 3, 112), (1, 515, 7, 32), (2, 300, 3, 128), (1, 77, 3, 7)],
                         ids=lambda s: "B%d_N%d_H%d_d%d" % s)
def test_state_and_apply_match_oracle(la, orc, shape, dtype):
    import torch

    B, N, H, d = shape
    q, k, v = gen(B, N, H, d, 2100 + N + d, dtype)
    S, z = orc.state(k, v)
    st = la.linattn_state(to_dev(k), to_dev(v))
    assert tuple(st.shape) == (B, H, d + 1, d) and st.dtype == torch.float32
    assert_state_close(to_f64(st), S, z, 1e-5, f"state {shape} {dtype}")
    # apply the ORACLE's state (rounded to fp32) so this checks the apply half alone
    W = np.ascontiguousarray(np.concatenate([S.swapaxes(-1, -2), z[..., None, :]], axis=-2), dtype=np.float32)
    o = la.linattn_apply(to_dev(q), torch.from_numpy(W).cuda(), EPS)
    ref = orc.apply_rows(q, W[..., :d, :].swapaxes(-1, -2).astype(np.float64).copy(), W[..., d, :].astype(np.float64).copy(),
                         EPS, np.arange(N))
    check(dtype, to_f64(o), ref, f"apply {shape} {dtype}")


@pytest.mark.parametrize("shape", [(2, 1000, 3, 112), (1, 515, 7, 32), (1, 4097, 2, 64), (1, 300, 2, 128)],
                         ids=lambda s: "B%d_N%d_H%d_d%d" % s)
def test_integer_inputs_give_bit_exact_state(la, orc, shape):
    """Inputs in {-2..2}: every partial sum is an integer < 2^24, so fp32 accumulation in any order
    must reproduce the oracle's state bit for bit (no tile lost, none counted twice)."""
    B, N, H, d = shape
    k = synth.smallint(shape[:1] + (N, H, d), 31, 2, 2)
    v = synth.smallint(shape[:1] + (N, H, d), 31, 3, 2)
    S, z = orc.state(k, v)
    st = to_f64(la.linattn_state(to_dev(k), to_dev(v)))
    assert np.array_equal(st[..., :d, :].swapaxes(-1, -2), S)
    assert np.array_equal(st[..., d, :], z)


def test_run_to_run_determinism(la):
    import torch

    q, k, v = (to_dev(x) for x in gen(2, 3000, 3, 112, 77, "bf16"))
    ws = la.new_workspace(q)
    o1 = la.linattn_forward(q, k, v, EPS, workspace=ws).clone()
    s1 = la.linattn_state(k, v, workspace=ws).clone()
    for _ in range(3):
        assert torch.equal(la.linattn_forward(q, k, v, EPS, workspace=ws), o1)
        assert torch.equal(la.linattn_state(k, v, workspace=ws), s1)


@pytest.mark.parametrize("d", [112, 32])
def test_constant_v_outputs_are_order_one(la, orc, d):
    """v_n = c: o = c*D/(D+eps).  Outputs of size ~1, so the absolute tolerance term is not vacuous."""
    B, N, H = 1, 700, 3
    q, k, _ = gen(B, N, H, d, 88, "bf16")
    c = synth.gauss((d,), 89, 3, dtype="bf16")
    v = np.broadcast_to(c, (B, N, H, d)).copy()
    o = to_f64(la.linattn_forward(to_dev(q), to_dev(k), to_dev(v), EPS))
    ref = orc.forward(q, k, v, EPS)
    assert_parity_bf16(o, ref, "constant V")
    cf = synth.bf16_bits_to_f32(c).astype(np.float64)
    live = np.abs(ref).sum(axis=-1) > 0
    assert np.allclose(o[live], np.broadcast_to(cf, o.shape)[live], rtol=1e-2, atol=1e-2)


@pytest.mark.parametrize("d", [112, 64])
def test_one_hot_features_give_segment_means(la, orc, d):
    B, N, H, C = 1, 900, 2, 5
    a = synth.index((N,), 91, 1, C)
    c = synth.index((N,), 91, 2, C)
    q = np.zeros((B, N, H, d), np.float32); q[0, np.arange(N), :, a * 3] = 1.0
    k = np.zeros((B, N, H, d), np.float32); k[0, np.arange(N), :, c * 3] = 2.0
    v = synth.bf16_bits_to_f32(synth.smallint((B, N, H, d), 91, 3, 4))
    qb, kb, vb = (synth.f32_to_bf16_bits(x) for x in (q, k, v))
    o = to_f64(la.linattn_forward(to_dev(qb), to_dev(kb), to_dev(vb), EPS))
    ref = orc.forward(qb, kb, vb, EPS)
    assert_parity_bf16(o, ref, "one-hot")
    cnt = np.bincount(c, minlength=C)
    mean = np.stack([np.bincount(c, weights=v[0, :, 0, j].astype(np.float64), minlength=C) / cnt for j in range(4)], 1)
    assert np.allclose(o[0, :, 0, :4], mean[a], rtol=1e-2, atol=1e-2)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_dead_queries_give_exact_zero(la, orc, dtype):
    """A query row with no positive entry has phi(q).z = 0: the output is 0/(0+eps) = 0, never NaN."""
    import torch

    B, N, H, d = 1, 300, 2, 112
    q, k, v = gen(B, N, H, d, 93, "f32")
    q[0, 5] = -np.abs(q[0, 5]); q[0, 128] = 0.0; q[0, 299, 1] = -1.0
    if dtype == "bf16":
        q, k, v = (synth.f32_to_bf16_bits(x) for x in (q, k, v))
    o = la.linattn_forward(to_dev(q), to_dev(k), to_dev(v), EPS)
    assert torch.isfinite(o.float()).all()
    assert (o[0, 5] == 0).all() and (o[0, 128] == 0).all() and (o[0, 299, 1] == 0).all()
    check(dtype, to_f64(o), orc.forward(q, k, v, EPS), "dead queries")
    # empty state: all keys non-positive -> every output is exactly zero
    k2 = -np.abs(synth.gauss((B, N, H, d), 94, 2, dtype="f32"))
    k2 = synth.f32_to_bf16_bits(k2) if dtype == "bf16" else k2
    o2 = la.linattn_forward(to_dev(q), to_dev(k2), to_dev(v), EPS)
    assert (o2 == 0).all()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_head_major_strides(la, orc, dtype):
    """[B,H,N,d] storage passed as a [B,N,H,d] view."""
    B, N, H, d = 2, 400, 3, 112
    q, k, v = gen(B, N, H, d, 95, dtype)
    ref = orc.forward(q, k, v, EPS)
    hm = lambda x: to_dev(np.ascontiguousarray(x.transpose(0, 2, 1, 3))).permute(0, 2, 1, 3)
    o = la.linattn_forward(hm(q), hm(k), hm(v), EPS)
    assert o.stride() == hm(q).stride()
    check(dtype, to_f64(o), ref, "head-major")


def test_zero_tokens_and_errors(la):
    import torch

    q = torch.zeros((1, 0, 2, 112), dtype=torch.bfloat16, device="cuda")
    o = la.linattn_forward(q, q.clone(), q.clone(), EPS)
    assert o.shape == q.shape
    st = la.linattn_state(q, q.clone())
    assert (st == 0).all()
    x = torch.zeros((1, 8, 2, 112), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(la.LinAttnError) as e:
        la.linattn_forward(x, x, x, EPS, out=x)  # aliasing
    assert e.value.status == -1
    big = torch.zeros((1, 8, 1, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(la.LinAttnError) as e:
        la.linattn_forward(big, big.clone(), big.clone(), EPS)
    assert e.value.status == -2
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(la.LinAttnError) as e:
        la.linattn_forward(x, x.clone(), x.clone(), EPS, workspace=ws)
    assert e.value.status == -4
    assert la.workspace_status(la.new_workspace(x)) == 0


@pytest.mark.parametrize("shape", [(1, 9000, 3, 112), (2, 8300, 2, 64), (1, 500, 2, 112)],
                         ids=lambda s: "B%d_N%d_H%d_d%d" % s)
def test_forward_from_host_buffers(la, orc, shape):
    """The host-buffer entry point (chunked upload of Q / download of O) gives the device path's bits."""
    import torch

    B, N, H, d = shape
    q, k, v = gen(B, N, H, d, 2300 + N, "bf16")
    pin = lambda bits: torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    qp, kp, vp = pin(q), pin(k), pin(v)
    op = torch.zeros_like(qp).pin_memory()
    hf = la.HostForward(B, N, H, d, torch.bfloat16, "cuda")
    for _ in range(2):  # twice: the staging area and the second stream are reused
        op.zero_()
        hf(qp, kp, vp, op, EPS)
        torch.cuda.synchronize()
        ref_dev = la.linattn_forward(to_dev(q), to_dev(k), to_dev(v), EPS)
        assert torch.equal(op.cuda(), ref_dev)
    assert_parity_bf16(to_f64(op), orc.forward(q, k, v, EPS), f"host forward {shape}")


def test_bounded_wait_reports_timeout_and_the_context_survives(la):
    """Every device-side wait is bounded.  A grid-barrier word that can never reach its target (the
    workspace's control block is required to start at zero; here it does not) makes the wait run out after
    about a second: the kernel returns, LINATTN_ERR_TIMEOUT is in the status word, nothing traps, and
    after re-initialising the workspace the same call works."""
    import torch

    q, k, v = (to_dev(x) for x in gen(1, 2000, 2, 112, 97, "bf16"))
    ws = la.new_workspace(q)
    good = la.linattn_state(k, v, workspace=ws).clone()
    ctrl = ws[:4096].view(torch.int32)
    ctrl[16] = 0x4000           # arrival count of the barrier word: the arrivals no longer carry into the generation
    la.linattn_state(k, v, workspace=ws)
    assert la.workspace_status(ws) == -6
    la.load_library().linattn_workspace_init(ws.data_ptr(), ws.numel(), torch.cuda.current_stream().cuda_stream)
    assert la.workspace_status(ws) == 0
    assert torch.equal(la.linattn_state(k, v, workspace=ws), good)


# Many units: how the persistent grid splits the work depends on the number of (batch, head) units U against
# the 148 SMs.  U = 60: two column CTAs per unit plus trailing CTAs, operand images in use; U = 100: one column
# CTA per unit plus trailing CTAs, images do not fit behind the records; U = 148: one CTA per unit, no trailing
# CTAs; U = 200: more units than CTAs, every CTA walks over several units.
@pytest.mark.parametrize("shape", [(3, 1500, 20, 112), (5, 700, 20, 112), (4, 600, 37, 112), (10, 400, 20, 112),
                                   (3, 900, 18, 128)], ids=lambda s: "B%d_N%d_H%d_d%d" % s)
def test_work_split_with_many_units(la, orc, shape):
    import torch

    B, N, H, d = shape
    q, k, v = gen(B, N, H, d, 2300 + B * H, "bf16")
    qd, kd, vd = to_dev(q), to_dev(k), to_dev(v)
    ws = la.new_workspace(qd)
    o = la.linattn_forward(qd, kd, vd, EPS, workspace=ws)
    check("bf16", to_f64(o), orc.forward(q, k, v, EPS), f"forward {shape}")
    assert torch.equal(o, la.linattn_forward(qd, kd, vd, EPS, workspace=ws))      # run-to-run determinism
    # the fused launch and the two separate launches sum the same records in the same order
    st = la.linattn_state(kd, vd, workspace=ws)
    assert torch.equal(o, la.linattn_apply(qd, st, EPS))
    # two cached steps over the halves: small integers make the cache exact, so both ways of reducing
    # (on top of the old cache, with or without operand images) must give the oracle's bits
    ki = synth.smallint((B, N, H, d), 2301, 2, 2)
    vi = synth.smallint((B, N, H, d), 2301, 3, 2)
    half = (N // 2 + 7) // 8 * 8
    cache = la.BlockLinCache(B, H, d, torch.bfloat16, "cuda", max_T_b=half, eps=EPS)
    outs = [cache.step(to_dev(np.ascontiguousarray(q[:, sl])), to_dev(np.ascontiguousarray(ki[:, sl])),
                       to_dev(np.ascontiguousarray(vi[:, sl]))) for sl in (slice(0, half), slice(half, N))]
    S, z = orc.state(ki, vi)
    got = to_f64(cache.state)
    assert np.array_equal(got[..., :d, :].swapaxes(-1, -2), S) and np.array_equal(got[..., d, :], z)
    ref = orc.block_masked(q, ki, vi, EPS, half)
    check("bf16", to_f64(torch.cat(outs, dim=1)), ref, f"two steps {shape}")
    assert la.workspace_status(cache.workspace) == 0


def _random_shapes(count, seed):
    rng = np.random.default_rng(seed)
    shapes = []
    while len(shapes) < count:
        d = int(rng.choice([32, 64, 112, 128]))
        B, H = int(rng.integers(1, 5)), int(rng.integers(1, 41))
        N = int(rng.integers(1, 3001))
        if B * H * N <= 150_000:
            shapes.append((B, N, H, d))
    return shapes


@pytest.mark.parametrize("shape", _random_shapes(16, 20250), ids=lambda s: "B%d_N%d_H%d_d%d" % s)
def test_seeded_random_shapes(la, orc, shape):
    """Shapes nobody picked by hand: forward against the oracle, the state of small-integer inputs bit for bit,
    and the same tokens as two cached steps of unequal length."""
    import torch

    B, N, H, d = shape
    q, k, v = gen(B, N, H, d, 2400 + N, "bf16")
    qd = to_dev(q)
    check("bf16", to_f64(la.linattn_forward(qd, to_dev(k), to_dev(v), EPS)), orc.forward(q, k, v, EPS), f"forward {shape}")
    ki = synth.smallint((B, N, H, d), 2401, 2, 2)
    vi = synth.smallint((B, N, H, d), 2401, 3, 2)
    S, z = orc.state(ki, vi)
    got = to_f64(la.linattn_state(to_dev(ki), to_dev(vi)))
    assert np.array_equal(got[..., :d, :].swapaxes(-1, -2), S) and np.array_equal(got[..., d, :], z)
    cut = max(1, N // 3)
    cache = la.BlockLinCache(B, H, d, torch.bfloat16, "cuda", max_T_b=max(cut, N - cut), eps=EPS)
    outs = [cache.step(to_dev(np.ascontiguousarray(q[:, sl])), to_dev(np.ascontiguousarray(ki[:, sl])),
                       to_dev(np.ascontiguousarray(vi[:, sl]))) for sl in (slice(0, cut), slice(cut, N)) if sl.stop > sl.start]
    got = to_f64(cache.state)
    assert np.array_equal(got[..., :d, :].swapaxes(-1, -2), S) and np.array_equal(got[..., d, :], z)
    # the second step's rows see everything: they equal the tail of the bidirectional result on the same inputs
    if N > cut:
        full = la.linattn_forward(qd, to_dev(ki), to_dev(vi), EPS)
        check("bf16", to_f64(outs[-1]), to_f64(full[:, cut:]).copy(), f"second step vs forward {shape}")
    assert la.workspace_status(cache.workspace) == 0


def test_hand_worked_example_on_the_gpu(la):
    """The hand-worked d = 2 example of tests/golden/ through the library itself (fp32 I/O path)."""
    import torch
    from parity_util import read_golden

    g = read_golden("eq2_eq3_hand_worked_d2.txt")
    q, k, v = (torch.from_numpy(g[n].reshape(1, 3, 1, 2).astype(np.float32)).cuda() for n in ("q", "k", "v"))
    st = to_f64(la.linattn_state(k, v))
    assert np.array_equal(st[0, 0, :2].T, g["S"]) and np.array_equal(st[0, 0, 2], g["z"][0])
    assert np.allclose(to_f64(la.linattn_forward(q, k, v, 0.0))[0, :, 0], g["o_bidirectional_eps0"], rtol=2e-7, atol=0)
    assert np.allclose(to_f64(la.linattn_forward(q, k, v, 0.5))[0, :, 0], g["o_bidirectional_eps_half"], rtol=2e-7, atol=0)
    cache = la.BlockLinCache(1, 1, 2, torch.float32, "cuda", max_T_b=2, eps=0.0)
    o12 = cache.step(q[:, :2].contiguous(), k[:, :2].contiguous(), v[:, :2].contiguous())
    o3 = cache.step(q[:, 2:].contiguous(), k[:, 2:].contiguous(), v[:, 2:].contiguous())
    assert np.allclose(to_f64(torch.cat([o12, o3], dim=1))[0, :, 0], g["o_blocks_12_3_eps0"], rtol=2e-7, atol=0)
