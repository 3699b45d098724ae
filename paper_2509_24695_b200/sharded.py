"""Token-sharded forms: one sequence (or one block of a stream) spread over several GPUs by tokens.

The state of Eq. 2, ``(sum_n phi(k_n)^T v_n, sum_n phi(k_n))``, and the running sums of Eq. 3 are sums over
tokens.  So every rank reduces the tokens it holds with the library's state kernel, ONE all-reduce (sum) of
``B*H*(d*d+d)`` floats (about 1 MB for 20 heads of 112) gives every rank the whole state in its own memory,
and every rank applies its own queries to it with the library's apply kernel.  Nothing else crosses the
link: Q, K, V and O stay where they are.

This module is rank logic only: which entry point runs on which shard, and where the collective sits.  The
arithmetic is in the library's kernels (``linattn_state`` / ``blocklin_shard_state`` and ``linattn_apply``)
and in the collective's sum.  The collective is ``torch.distributed.all_reduce`` on the given process group
(NCCL on GPUs); it reads and writes this rank's own buffer, and no kernel of the library is ever handed
another GPU's memory.

The kernels and the collective are passed in as callables so that the rank logic can be exercised on CPU
ranks (``gloo``) with stand-ins; the defaults are the library's entry points.
"""
from __future__ import annotations

import ctypes

__all__ = ["shard_bounds", "linattn_forward_token_sharded", "TokenShardedCache"]


def shard_bounds(n_tokens: int, world: int, rank: int, multiple: int = 1) -> tuple[int, int]:
    """Token range ``[lo, hi)`` of `rank` when `n_tokens` are dealt to `world` ranks in contiguous, nearly equal
    pieces whose starts are multiples of `multiple` (the last rank takes the remainder)."""
    if world < 1 or not 0 <= rank < world or n_tokens < 0 or multiple < 1:
        raise ValueError("bad shard request")
    units = -(-n_tokens // multiple)
    lo = min(n_tokens, (units * rank // world) * multiple)
    hi = min(n_tokens, (units * (rank + 1) // world) * multiple)
    return lo, hi


def _all_reduce_sum(t, group):
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return t


def linattn_forward_token_sharded(q, k, v, eps: float = 1e-6, group=None, out=None, workspace=None,
                                  state_fn=None, apply_fn=None, all_reduce=_all_reduce_sum):
    """Eq. 2 over a sequence whose tokens are split over the ranks of `group`.

    q, k, v: this rank's tokens ``[B, N_local, H, d]`` (shards may differ in length, and may be empty).  Returns
    this rank's rows of O and the whole sequence's state (identical on every rank).
    """
    if state_fn is None or apply_fn is None:
        import paper_2509_24695_b200 as la

        ws = la.new_workspace(k) if workspace is None else workspace
        state_fn = state_fn or (lambda k_, v_: la.linattn_state(k_, v_, workspace=ws))
        apply_fn = apply_fn or (lambda q_, st: la.linattn_apply(q_, st, eps, out=out, workspace=ws))
    state = state_fn(k, v)               # this shard's partial sums (zeros for an empty shard)
    state = all_reduce(state, group)     # the one exchange: ~1 MB, summed into this rank's own buffer
    return apply_fn(q, state), state


class TokenShardedCache:
    """The constant-memory cache of Eq. 3 when every block's tokens are split over the ranks of `group`.

    Every rank keeps a full copy of the cache (it is ~1 MB) and they stay bit-identical: a step all-reduces the
    ranks' shares of the NEW cache, where rank 0's share includes the old cache, so the sum over ranks is
    ``cache + state(block)`` and every rank adopts the same bits.

    `cache` is a ``BlockLinCache``.  The three local operations default to the library's entry points
    (``blocklin_shard_state``, ``blocklin_shard_commit``, ``linattn_apply``); CPU tests of the rank logic pass
    stand-ins: ``share_fn(k, v, include_cache) -> state tensor``, ``commit_fn(state, block_tokens)``,
    ``apply_fn(q, out) -> o``.
    """

    def __init__(self, cache, group=None, all_reduce=_all_reduce_sum, rank=None, share_fn=None, commit_fn=None,
                 apply_fn=None):
        self.cache, self.group, self._all_reduce = cache, group, all_reduce
        if rank is None:
            import torch.distributed as dist

            live = dist.is_available() and dist.is_initialized()
            rank = dist.get_rank(group) if live else 0
        self.rank = rank
        self._share = None
        self._share_fn = share_fn or self._lib_share
        self._commit_fn = commit_fn or self._lib_commit
        self._apply_fn = apply_fn or self._lib_apply

    def _lib_share(self, k, v, include_cache):
        import paper_2509_24695_b200 as la
        import torch

        c = self.cache
        c._check_layout(k)
        if self._share is None:
            self._share = torch.empty_like(c.state)
        la._check(la.load_library().blocklin_shard_state(c._handle, k.shape[1], la._ptr(k), la._ptr(v), la._ptr(self._share),
                                                         1 if include_cache else 0, la._stream(k)), "blocklin_shard_state")
        return self._share

    def _lib_commit(self, state, block_tokens):
        import paper_2509_24695_b200 as la

        c = self.cache
        la._check(la.load_library().blocklin_shard_commit(c._handle, la._ptr(state), ctypes.c_int64(block_tokens),
                                                          la._stream(state)), "blocklin_shard_commit")

    def _lib_apply(self, q, out):
        import paper_2509_24695_b200 as la

        c = self.cache
        return la.linattn_apply(q, c.state, c.eps, out=out, workspace=c.workspace)

    def step(self, q, k, v, block_tokens: int, out=None):
        """One block: q, k, v are this rank's tokens of it (possibly none), block_tokens the block's length over
        all ranks.  Returns this rank's rows of the block's output (None when q is None: absorb only)."""
        share = self._share_fn(k, v, self.rank == 0)     # rank 0's share carries the old cache
        share = self._all_reduce(share, self.group)      # the one exchange of the step
        self._commit_fn(share, block_tokens)             # every rank adopts the same new cache
        return None if q is None else self._apply_fn(q, out)
