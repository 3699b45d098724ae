"""Seeded random walks over the block-causal API against the oracle.

Each case draws a shape (batch, heads, head dim, dtype) and a sequence of blocks of random lengths, and at every block
picks what to do with it: a committed step, a read-only step before it, an absorb-only step, or a step whose tokens
are split over two "ranks" (two caches in one process; their shares are summed here on the host the way an
all-reduce would, which is the one piece of arithmetic this test does itself).  One walk uses the plain form, one
the form with rotary factors.  Outputs are compared with the oracle's block-masked forms, the cache with the
oracle's cache, and the cache size must never change.
"""
import ctypes

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


def draw_case(seed):
    rng = np.random.default_rng(seed)
    d = int(rng.choice([32, 64, 112, 112, 128, 40, 6]))
    dtype = "f32" if rng.random() < 0.25 else "bf16"
    B, H = int(rng.integers(1, 4)), int(rng.integers(1, 24))
    n_blocks = int(rng.integers(2, 6))
    lens = [int(rng.integers(1, 700)) for _ in range(n_blocks)]
    while B * H * sum(lens) > 60_000:
        lens = [max(1, n // 2) for n in lens]
    return rng, B, H, d, dtype, lens


def state_close(got, S, z, rel, what):
    d = S.shape[-1]
    for g, r, name in ((got[..., :d, :].swapaxes(-1, -2), S, "S"), (got[..., d, :], z, "z")):
        rms = np.sqrt((r ** 2).mean(axis=tuple(range(2, r.ndim)), keepdims=True))
        assert (np.abs(g - r) <= rel * (np.abs(r) + rms)).all(), f"{what}: {name}"


@pytest.mark.parametrize("seed", range(9100, 9112))
def test_random_walk_plain(la, orc, seed):
    import torch

    rng, B, H, d, dtype, lens = draw_case(seed)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    check = assert_parity_bf16 if dtype == "bf16" else assert_parity_f32
    N = sum(lens)
    q, k, v = (synth.gauss((B, N, H, d), seed, t, dtype=dtype) for t in (1, 2, 3))
    cache = la.BlockLinCache(B, H, d, tdt, "cuda", max_T_b=max(lens), eps=EPS)
    other = la.BlockLinCache(B, H, d, tdt, "cuda", max_T_b=max(lens), eps=EPS)     # the second "rank" of sharded steps
    lib = la.load_library()
    S, z = orc.new_cache(B, H, d)
    bytes0 = cache.info()["state_bytes"]
    n0 = 0
    for i, T in enumerate(lens):
        sl = slice(n0, n0 + T)
        blk_h = [np.ascontiguousarray(x[:, sl]) for x in (q, k, v)]
        blk = [to_dev(x) for x in blk_h]
        mode = rng.choice(["step", "peek+step", "absorb", "sharded"])
        what = f"seed {seed} block {i} ({mode}, T={T}, B{B} H{H} d{d} {dtype})"
        if mode == "peek+step":
            before = cache.state.clone()
            o_peek = cache.peek(*blk)
            assert torch.equal(cache.state, before)
            o = cache.step(*blk)
            assert torch.equal(o, o_peek)
        elif mode == "absorb":
            assert cache.step(None, blk[1], blk[2]) is None
            o = None
        elif mode == "sharded":
            cut = int(rng.integers(0, T + 1))                       # rank 0 holds [0, cut), rank 1 the rest (either may be empty)
            other.state.copy_(cache.state)                          # every rank holds the same cache
            shares = []
            for c, (a, b), inc in ((cache, (0, cut), 1), (other, (cut, T), 0)):
                share = torch.empty_like(c.state)
                kk, vv = blk[1][:, a:b].contiguous(), blk[2][:, a:b].contiguous()
                st = lib.blocklin_shard_state(c._handle, b - a, kk.data_ptr() if b > a else None, vv.data_ptr() if b > a else None,
                                              share.data_ptr(), inc, ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
                assert st == 0, what
                shares.append(share)
            total = shares[0] + shares[1]                           # what the all-reduce would leave on every rank
            outs = []
            for c, (a, b) in ((cache, (0, cut)), (other, (cut, T))):
                assert lib.blocklin_shard_commit(c._handle, total.data_ptr(), T, ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)) == 0
                outs.append(la.linattn_apply(blk[0][:, a:b].contiguous(), c.state, EPS, workspace=c.workspace))
            o = torch.cat(outs, dim=1)
            assert torch.equal(cache.state, other.state)
        else:
            o = cache.step(*blk)
        ref = orc.block_step((S, z), *blk_h, EPS)                   # the oracle commits the block and reads it
        if o is not None:
            check(to_f64(o), ref, what)
        state_close(to_f64(cache.state), S, z, 1e-5, what)
        assert cache.info()["state_bytes"] == bytes0 == B * H * (d * d + d) * 4
        n0 += T
    assert cache.info()["blocks_seen"] == len(lens) and cache.info()["tokens_seen"] == N and cache.status() == 0
    # the whole walk equals the one-shot block-masked form only for equal blocks; what always holds: the last block's
    # queries saw everything, so its rows equal the bidirectional forward's
    if o is not None:
        full = orc.forward(q, k, v, EPS)
        check(to_f64(o), full[:, N - lens[-1]:], f"seed {seed}: last block vs bidirectional forward")


@pytest.mark.parametrize("seed", range(9200, 9210))
def test_random_walk_rotary(la, orc, seed):
    import torch

    rng, B, H, d, dtype, lens = draw_case(seed)
    if d % 2:
        d += 1
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    check = assert_parity_f32
    if dtype == "bf16":   # the tensor-core path rounds the rotated queries and keys to bf16 as well
        check = lambda got, ref, what: assert_parity_bf16(got, ref, what, rms_rel=1.5e-2 if d in (32, 64, 112, 128) else 1e-2)
    N = sum(lens)
    q, k, v = (synth.gauss((B, N, H, d), seed, t, dtype=dtype) for t in (1, 2, 3))
    theta = synth.gauss((N, d // 2), seed, 7, dtype="f32").astype(np.float64) * 3.0
    table = la.rope_pack(to_dev(np.cos(theta).astype(np.float32)), to_dev(np.sin(theta).astype(np.float32)))
    packed = table.cpu().numpy().astype(np.float64)
    cs, sn = packed[..., 0], packed[..., 1]
    cache = la.BlockLinCache(B, H, d, tdt, "cuda", max_T_b=max(lens), eps=EPS)
    ocache = orc.new_cache(B, H, d)
    n0 = 0
    for i, T in enumerate(lens):
        sl = slice(n0, n0 + T)
        blk_h = [np.ascontiguousarray(x[:, sl]) for x in (q, k, v)]
        blk = [to_dev(x) for x in blk_h]
        tab = table[sl].contiguous()
        mode = rng.choice(["step", "peek+step", "absorb"])
        what = f"seed {seed} block {i} ({mode}, T={T}, B{B} H{H} d{d} {dtype})"
        o = None
        if mode == "peek+step":
            before = cache.state.clone()
            o_peek = cache.peek_rope(*blk, tab)
            assert torch.equal(cache.state, before)
            o = cache.step_rope(*blk, tab)
            assert torch.equal(o, o_peek)
        elif mode == "absorb":
            assert cache.step_rope(None, blk[1], blk[2], tab) is None
        else:
            o = cache.step_rope(*blk, tab)
        ref = orc.rope_block_step(ocache, *blk_h, cs[sl], sn[sl], EPS)
        if o is not None:
            check(to_f64(o), ref, what)
        # the tensor-core path (bf16, d = 32, 64, 112 or 128) rounds the rotated keys to bf16 before the MMA
        state_close(to_f64(cache.state), *ocache, 1e-2 if (dtype == "bf16" and d in (32, 64, 112, 128)) else 1e-5, what)
        n0 += T
    assert cache.info()["blocks_seen"] == len(lens) and cache.status() == 0
