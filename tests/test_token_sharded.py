"""The token-sharded form: a sequence (or each block of a stream) split by tokens over two ranks.

Eq. 2's state and Eq. 3's running sums are sums over tokens, so each rank reduces its own shard, one all-reduce
(sum) of the state follows, and each rank applies its own queries.  Two tests:

 * CPU, two `gloo` ranks: the rank logic alone (which shard goes where, where the collective sits, that rank 0
   alone contributes the old cache), with the oracle standing in for the kernels.  Small-integer inputs make
   every sum exact, so the result must equal the oracle's whole-sequence result bit for bit.
 * GPU (marked gpu), two `gloo` ranks that share the one visible GPU: the library's kernels on each shard.  The
   ranks take turns on the GPU (a barrier after every launch sequence), so no kernel of one rank ever runs
   beside, or waits for, a kernel of the other.
"""
import json
import os
import subprocess
import sys
import textwrap

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

COMMON = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r); sys.path.insert(0, os.path.join(%r, "tests"))
    import numpy as np, torch, torch.distributed as dist
    import oracle, synth
    from paper_2509_24695_b200 import sharded
    import datetime
    dist.init_process_group("gloo", timeout=datetime.timedelta(seconds=90))   # a rank that fails ends the other soon
    rank, world = dist.get_rank(), dist.get_world_size()
    orc = oracle.default()
    B, N, H, d, T_b, eps = 2, 1130, 3, %d, 400, 1e-6
    q = synth.gauss((B, N, H, d), 7001, 1)
    k, v = synth.smallint((B, N, H, d), 7001, 2, 2), synth.smallint((B, N, H, d), 7001, 3, 2)
""")

CPU_WORKER = COMMON % (ROOT, ROOT, 16) + textwrap.dedent("""
    def pack(S, z):                      # one tensor per state, so that ONE all-reduce moves it
        return torch.from_numpy(np.concatenate([S.reshape(B, H, -1), z], axis=2))
    def unpack(t):
        a = t.numpy()
        return np.ascontiguousarray(a[..., :d * d]).reshape(B, H, d, d), np.ascontiguousarray(a[..., d * d:])
    state_fn = lambda k_, v_: pack(*orc.state(k_, v_))
    apply_fn = lambda q_, st: orc.apply_rows(q_, *unpack(st), eps, np.arange(q_.shape[1]))
    lo, hi = sharded.shard_bounds(N, world, rank, multiple=64)
    sl = lambda x: np.ascontiguousarray(x[:, lo:hi])
    o, st = sharded.linattn_forward_token_sharded(sl(q), sl(k), sl(v), eps, state_fn=state_fn, apply_fn=apply_fn)
    S, z = orc.state(k, v)
    ok_state = bool(np.array_equal(unpack(st)[0], S) and np.array_equal(unpack(st)[1], z))
    ok_rows = bool(np.array_equal(o, orc.forward(q, k, v, eps)[:, lo:hi]))
    # an empty shard: rank 1 holds nothing, rank 0 everything
    lo2, hi2 = (0, N) if rank == 0 else (N, N)
    o2, st2 = sharded.linattn_forward_token_sharded(np.ascontiguousarray(q[:, lo2:hi2]), np.ascontiguousarray(k[:, lo2:hi2]),
                                                    np.ascontiguousarray(v[:, lo2:hi2]), eps, state_fn=state_fn, apply_fn=apply_fn)
    ok_empty = bool(torch.equal(st2, st) and o2.shape[1] == hi2 - lo2)
    # block by block with a replicated cache: rank 0's share carries the old cache, every rank adopts the sum
    class Box: pass
    box = Box(); box.S, box.z = orc.new_cache(B, H, d)
    def share_fn(k_, v_, include_cache):
        S_, z_ = orc.state(k_, v_)
        return pack(S_ + box.S, z_ + box.z) if include_cache else pack(S_, z_)
    def commit_fn(st_, tokens): box.S, box.z = unpack(st_)
    tsc = sharded.TokenShardedCache(None, share_fn=share_fn, commit_fn=commit_fn,
                                    apply_fn=lambda q_, out: orc.apply_rows(q_, box.S, box.z, eps, np.arange(q_.shape[1])))
    ref = orc.block_masked(q, k, v, eps, T_b)
    ok_steps = True
    for n0 in range(0, N, T_b):
        n1 = min(n0 + T_b, N)
        a, b = sharded.shard_bounds(n1 - n0, world, rank, multiple=128)
        ob = tsc.step(*(np.ascontiguousarray(x[:, n0 + a:n0 + b]) for x in (q, k, v)), block_tokens=n1 - n0)
        ok_steps = ok_steps and bool(np.array_equal(ob, ref[:, n0 + a:n0 + b]))
    ok_steps = ok_steps and bool(np.array_equal(box.S, S) and np.array_equal(box.z, z))
    print(json.dumps({"rank": rank, "lo": lo, "hi": hi, "ok_state": ok_state, "ok_rows": ok_rows, "ok_empty": ok_empty,
                      "ok_steps": ok_steps}))
    dist.destroy_process_group()
""")

GPU_WORKER = COMMON % (ROOT, ROOT, 112) + textwrap.dedent("""
    import paper_2509_24695_b200 as la
    from parity_util import assert_parity_bf16, to_dev, to_f64
    torch.cuda.set_device(0)
    def my_turn(fn):                     # the ranks take turns on the one GPU: launch, finish, then the other
        out = None
        for r in range(world):
            if r == rank:
                out = fn(); torch.cuda.synchronize()
            dist.barrier()
        return out
    def all_reduce_via_host(t, group):   # gloo sums on the host; the result lands in this rank's own buffer
        torch.cuda.synchronize()
        h = t.cpu(); dist.all_reduce(h, op=dist.ReduceOp.SUM, group=group); t.copy_(h); torch.cuda.synchronize()
        return t
    lo, hi = sharded.shard_bounds(N, world, rank, multiple=128)
    sl = lambda x: to_dev(np.ascontiguousarray(x[:, lo:hi]))
    qd, kd, vd = sl(q), sl(k), sl(v)
    ws = la.new_workspace(kd)
    res = {"rank": rank, "lo": lo, "hi": hi}
    # whole sequence, bidirectional
    st = my_turn(lambda: la.linattn_state(kd, vd, workspace=ws))
    all_reduce_via_host(st, None)
    o = my_turn(lambda: la.linattn_apply(qd, st, eps, workspace=ws))
    S, z = orc.state(k, v)
    g = to_f64(st)
    res["state_exact"] = bool(np.array_equal(g[..., :d, :].swapaxes(-1, -2), S) and np.array_equal(g[..., d, :], z))
    assert_parity_bf16(to_f64(o), orc.forward(q, k, v, eps)[:, lo:hi], "token-sharded forward")
    # block by block: every block's tokens split over the ranks, the cache replicated
    cache = la.BlockLinCache(B, H, d, torch.bfloat16, "cuda", max_T_b=T_b, eps=eps)
    lib_ops = sharded.TokenShardedCache(cache)
    tsc = sharded.TokenShardedCache(cache, all_reduce=all_reduce_via_host,       # each local half in this rank's turn
                                    share_fn=lambda k_, v_, inc: my_turn(lambda: lib_ops._lib_share(k_, v_, inc)),
                                    commit_fn=lambda st_, n_: my_turn(lambda: lib_ops._lib_commit(st_, n_)),
                                    apply_fn=lambda q_, out: my_turn(lambda: lib_ops._lib_apply(q_, out)))
    ref = orc.block_masked(q, k, v, eps, T_b)
    ocache = orc.new_cache(B, H, d)
    for n0 in range(0, N, T_b):
        n1 = min(n0 + T_b, N)
        a, b = sharded.shard_bounds(n1 - n0, world, rank, multiple=128)
        blk = [to_dev(np.ascontiguousarray(x[:, n0 + a:n0 + b])) for x in (q, k, v)]
        ob = tsc.step(*blk, block_tokens=n1 - n0)
        torch.cuda.synchronize()
        assert_parity_bf16(to_f64(ob), ref[:, n0 + a:n0 + b], "token-sharded block step at %d" % n0)
        orc.block_step(ocache, np.ascontiguousarray(q[:, n0:n1]), np.ascontiguousarray(k[:, n0:n1]), np.ascontiguousarray(v[:, n0:n1]), eps, want_o=False)
        g = to_f64(cache.state)
        assert np.array_equal(g[..., :d, :].swapaxes(-1, -2), ocache[0]) and np.array_equal(g[..., d, :], ocache[1])
    res["info"] = cache.info()
    res["status"] = cache.status()
    # every rank holds the same cache bits
    mine = cache.state.cpu(); other = mine.clone(); dist.broadcast(other, src=0)
    res["cache_same_on_all_ranks"] = bool(torch.equal(mine, other))
    print(json.dumps(res))
    dist.destroy_process_group()
""")


def run_ranks(tmp_path, text, timeout):
    script = tmp_path / "worker.py"
    script.write_text(text)
    port = 31500 + os.getpid() % 2000
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=timeout) for p in procs]
    for p, (so, se) in zip(procs, outs):
        assert p.returncode == 0, se[-3000:]
    return [json.loads(so.strip().splitlines()[-1]) for so, _ in outs]


def test_shard_bounds():
    from paper_2509_24695_b200.sharded import shard_bounds

    for n, world, mult in ((1130, 2, 64), (32760, 8, 128), (5, 4, 1), (0, 3, 128), (100, 3, 128)):
        pieces = [shard_bounds(n, world, r, mult) for r in range(world)]
        assert pieces[0][0] == 0 and pieces[-1][1] == n
        assert all(a[1] == b[0] for a, b in zip(pieces[:-1], pieces[1:]))        # contiguous, nothing lost or doubled
        assert all(lo % mult == 0 or lo == n for lo, _ in pieces)
    with pytest.raises(ValueError):
        shard_bounds(10, 2, 2)


def test_two_gloo_ranks_rank_logic_with_the_oracle_as_kernels(tmp_path):
    outs = run_ranks(tmp_path, CPU_WORKER, 300)
    assert sorted((o["lo"], o["hi"]) for o in outs) == [(0, 576), (576, 1130)]
    for o in outs:
        assert o["ok_state"] and o["ok_rows"] and o["ok_empty"] and o["ok_steps"], o


@pytest.mark.gpu
def test_two_ranks_on_one_gpu_match_the_oracle(tmp_path):
    outs = run_ranks(tmp_path, GPU_WORKER, 400)
    for o in outs:
        assert o["state_exact"] and o["cache_same_on_all_ranks"] and o["status"] == 0, o
        assert o["info"] == {"blocks_seen": 3, "tokens_seen": 1130, "state_bytes": 2 * 3 * (112 * 112 + 112) * 4}
