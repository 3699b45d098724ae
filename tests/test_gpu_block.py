"""GPU parity of the block-causal form with the constant-memory cache (Eq. 3, Algorithm 1's cache
update) against the oracle's one-shot block-masked computation."""
import numpy as np
import pytest

import synth
from parity_util import assert_parity_bf16, assert_parity_f32, assert_state_close, to_dev, to_f64

pytestmark = pytest.mark.gpu

EPS = 1e-6


@pytest.fixture(scope="module")
def la():
    import torch

    assert torch.cuda.is_available()
    import paper_2509_24695_b200 as la

    la.load_library()
    return la


def gen(B, N, H, d, seed, dtype):
    return tuple(synth.gauss((B, N, H, d), seed, t, dtype=dtype) for t in (1, 2, 3))


def tdtype(dtype):
    import torch

    return torch.bfloat16 if dtype == "bf16" else torch.float32


CASES = [
    # B, H, d, T_b, n_blocks
    (1, 3, 112, 520, 7),   # config 4 in miniature: 7 blocks, several tiles each, ragged
    (2, 2, 112, 129, 4),
    (1, 5, 32, 200, 3),
    (1, 2, 64, 64, 5),
    (2, 1, 128, 150, 3),
    (1, 2, 24, 50, 4),
]


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("case", CASES, ids=lambda c: "B%d_H%d_d%d_T%d_M%d" % c)
def test_steps_equal_block_masked_oracle(la, orc, case, dtype):
    import torch

    B, H, d, T_b, M = case
    N = T_b * M
    q, k, v = gen(B, N, H, d, 3000 + T_b + d, dtype)
    ref = orc.block_masked(q, k, v, EPS, T_b)
    S, z = orc.state(k, v)
    check = assert_parity_bf16 if dtype == "bf16" else assert_parity_f32

    cache = la.BlockLinCache(B, H, d, tdtype(dtype), "cuda", max_T_b=T_b, eps=EPS)
    cache_ws_bytes = cache.workspace.numel()
    bytes0 = cache.info()["state_bytes"]
    assert bytes0 == B * H * (d * d + d) * 4 == cache.state.numel() * 4
    outs = []
    for b in range(M):
        sl = slice(b * T_b, (b + 1) * T_b)
        qb, kb, vb = (to_dev(np.ascontiguousarray(x[:, sl])) for x in (q, k, v))
        outs.append(cache.step(qb, kb, vb))
        info = cache.info()
        # the cache never grows with the number of blocks (Table 1)
        assert info == {"blocks_seen": b + 1, "tokens_seen": (b + 1) * T_b, "state_bytes": bytes0}
    stepped = torch.cat(outs, dim=1)
    check(to_f64(stepped), ref, f"steps {case} {dtype}")
    # final cache == state of the whole sequence
    assert_state_close(to_f64(cache.state), S, z, 1e-5, "final cache")
    # last block's output == tail of the bidirectional forward over everything
    full = la.linattn_forward(to_dev(q), to_dev(k), to_dev(v), EPS)
    check(to_f64(stepped[:, -T_b:]), to_f64(full[:, -T_b:]).copy(), "last block vs bidirectional")

    # prefill in one call == the same steps, bit for bit, and leaves the same cache
    final_state = cache.state.clone()
    cache.reset()
    assert cache.info()["blocks_seen"] == 0 and (cache.state == 0).all()
    o_pre = cache.prefill(to_dev(q), to_dev(k), to_dev(v), M)
    assert torch.equal(o_pre, stepped)
    assert torch.equal(cache.state, final_state)
    assert cache.info()["blocks_seen"] == M
    cache.close()

    # a cache with room for all M blocks takes them together (one state pass, a prefix over the blocks, one
    # apply pass): same mathematics, sums associated differently, so the oracle is the reference again
    big = la.BlockLinCache(B, H, d, tdtype(dtype), "cuda", max_T_b=T_b, eps=EPS, prefill_blocks=M)
    assert big.workspace.numel() >= cache_ws_bytes
    launches0 = la.kernel_launches()
    o_all = big.prefill(to_dev(q), to_dev(k), to_dev(v), M)
    assert la.kernel_launches() - launches0 <= 4   # state (+ its reduce), prefix, apply: not one set per block
    check(to_f64(o_all), ref, f"prefill all blocks {case} {dtype}")
    assert_state_close(to_f64(big.state), S, z, 1e-5, "cache after prefill of all blocks")
    assert big.info() == {"blocks_seen": M, "tokens_seen": N, "state_bytes": bytes0}
    # and it continues from a non-empty cache: a second prefill of the same blocks doubles the state
    o_again = big.prefill(to_dev(q), to_dev(k), to_dev(v), M)
    assert_state_close(to_f64(big.state), 2 * S, 2 * z, 1e-5, "cache after two prefills")
    S1, z1 = orc.state(np.ascontiguousarray(k[:, :T_b]), np.ascontiguousarray(v[:, :T_b]))
    first = orc.apply_rows(np.ascontiguousarray(q[:, :T_b]), S + S1, z + z1, EPS, np.arange(T_b))
    check(to_f64(o_again[:, :T_b]), first, "first block of the second prefill")
    assert la.workspace_status(big.workspace) == 0
    big.close()


def test_single_block_equals_forward(la):
    import torch

    B, N, H, d = 1, 700, 3, 112
    q, k, v = (to_dev(x) for x in gen(B, N, H, d, 3100, "bf16"))
    cache = la.BlockLinCache(B, H, d, torch.bfloat16, "cuda", max_T_b=N, eps=EPS)
    o = cache.step(q, k, v)
    assert torch.equal(o, la.linattn_forward(q, k, v, EPS))
    assert torch.equal(cache.state, la.linattn_state(k, v))


def test_checkpoint_restore_and_absorb_only(la, orc):
    """The state tensor is the whole generation state: snapshot, continue, restore, continue again."""
    import torch

    B, H, d, T_b, M = 1, 2, 112, 300, 5
    q, k, v = gen(B, T_b * M, H, d, 3200, "bf16")
    blk = lambda x, b: to_dev(np.ascontiguousarray(x[:, b * T_b:(b + 1) * T_b]))
    cache = la.BlockLinCache(B, H, d, torch.bfloat16, "cuda", max_T_b=T_b, eps=EPS)
    for b in range(2):
        cache.step(None, blk(k, b), blk(v, b))  # absorb context without producing outputs
    snap = cache.state.clone()
    first = [cache.step(blk(q, b), blk(k, b), blk(v, b)).clone() for b in range(2, M)]
    cache.state.copy_(snap)
    again = [cache.step(blk(q, b), blk(k, b), blk(v, b)) for b in range(2, M)]
    for a, b_ in zip(first, again):
        assert torch.equal(a, b_)
    ref = orc.block_masked(q, k, v, EPS, T_b)
    assert_parity_bf16(to_f64(torch.cat(again, dim=1)), ref[:, 2 * T_b:], "after absorb-only prefix")


def test_ragged_last_block(la, orc):
    import torch

    B, H, d, T_b = 1, 2, 112, 256
    N = 3 * T_b + 77
    q, k, v = gen(B, N, H, d, 3300, "bf16")
    ref = orc.block_masked(q, k, v, EPS, T_b)
    cache = la.BlockLinCache(B, H, d, torch.bfloat16, "cuda", max_T_b=T_b, eps=EPS)
    outs = []
    for n0 in range(0, N, T_b):
        sl = slice(n0, min(n0 + T_b, N))
        outs.append(cache.step(*(to_dev(np.ascontiguousarray(x[:, sl])) for x in (q, k, v))))
    assert_parity_bf16(to_f64(torch.cat(outs, dim=1)), ref, "ragged last block")
    assert cache.info()["tokens_seen"] == N


def test_block_errors(la):
    import torch

    cache = la.BlockLinCache(1, 2, 112, torch.bfloat16, "cuda", max_T_b=64, eps=EPS)
    x = torch.zeros((1, 64, 2, 112), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(la.LinAttnError) as e:
        cache.step(x, x, x, out=x)
    assert e.value.status == -1
    big = torch.zeros((1, 100000, 2, 112), dtype=torch.bfloat16, device="cuda")
    try:
        cache.step(big, big.clone(), big.clone())
    except la.LinAttnError as err:  # a block beyond max_T_b may or may not fit the workspace
        assert err.status == -4
    assert cache.step(x[:, :0], x[:, :0].clone(), x[:, :0].clone()).shape[1] == 0
    assert cache.info()["blocks_seen"] in (0, 1)


@pytest.mark.parametrize("dtype,d", [("bf16", 112), ("bf16", 64), ("f32", 112), ("bf16", 40)])
def test_denoise_loop_reads_without_committing(la, orc, dtype, d):
    """Algorithm 1: every denoising step of a block reads the cache together with the (noisy) block itself
    but leaves the cache as it was; only the clean block is committed, once."""
    import torch

    B, H, T_b, M, T = 1, 3, 300, 3, 3
    check = assert_parity_bf16 if dtype == "bf16" else assert_parity_f32
    cache = la.BlockLinCache(B, H, d, tdtype(dtype), "cuda", max_T_b=T_b, eps=EPS)
    S, z = orc.new_cache(B, H, d)
    for blk in range(M):
        before = cache.state.clone()
        for j in range(T):  # noisy versions of the block: other values each time
            q, k, v = gen(B, T_b, H, d, 3400 + 10 * blk + j, dtype)
            o = cache.peek(to_dev(q), to_dev(k), to_dev(v))
            ref = orc.block_step((S.copy(), z.copy()), q, k, v, EPS)   # the oracle's step on a COPY of its cache
            check(to_f64(o), ref, f"peek block {blk} step {j}")
            assert torch.equal(cache.state, before), "a read-only step changed the cache"
            assert cache.info()["blocks_seen"] == blk
        q, k, v = gen(B, T_b, H, d, 3500 + blk, dtype)               # the clean block
        o_peek = cache.peek(to_dev(q), to_dev(k), to_dev(v))
        o_step = cache.step(to_dev(q), to_dev(k), to_dev(v))
        assert torch.equal(o_peek, o_step)                            # same arithmetic, committed or not
        orc.block_step((S, z), q, k, v, EPS, want_o=False)
        assert_state_close(to_f64(cache.state), S, z, 1e-5, f"cache after block {blk}")
    assert cache.info()["blocks_seen"] == M


def test_steps_replay_from_a_cuda_graph(la):
    """A run of cached steps captured into a CUDA graph and replayed gives the bits of the same steps launched one
    by one (every call only enqueues work on the stream it is given; nothing is allocated or synchronised)."""
    import ctypes

    import torch

    B, H, d, T_b, M = 1, 4, 112, 520, 3
    q, k, v = (to_dev(x) for x in gen(B, T_b * M, H, d, 3300, "bf16"))
    blocks = [tuple(t[:, i * T_b:(i + 1) * T_b].contiguous() for t in (q, k, v)) for i in range(M)]
    cache = la.BlockLinCache(B, H, d, torch.bfloat16, "cuda", max_T_b=T_b, eps=EPS)
    eager = [cache.step(*blk) for blk in blocks]          # also the warm-up a capture needs
    final = cache.state.clone()
    outs = [torch.empty_like(o) for o in eager]
    lib = la.load_library()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        cache.reset()
        with torch.cuda.graph(graph, stream=side):
            handle = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
            for (qb, kb, vb), ob in zip(blocks, outs):
                assert lib.blocklin_step(cache._handle, T_b, qb.data_ptr(), kb.data_ptr(), vb.data_ptr(), ob.data_ptr(),
                                         handle) == 0
        for _ in range(2):                                  # replay twice: the second one starts from a reset cache too
            cache.reset()
            graph.replay()
            side.synchronize()
            assert all(torch.equal(a, b) for a, b in zip(outs, eager))
            assert torch.equal(cache.state, final)
    torch.cuda.current_stream().wait_stream(side)
    assert la.workspace_status(cache.workspace) == 0
