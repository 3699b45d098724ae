"""Out-of-bounds evidence: every buffer the library writes sits between two guard bands that must stay intact.

Outputs, caches, states and workspaces are carved out of one byte pool with a band of a fixed pattern on both
sides.  After every call the bands are compared with the pattern: a TMA store that runs past a ragged tail, a
partial record written beyond the workspace, or a cache frame written at the wrong batch offset would land in a
band (a neighbouring torch allocation would hide it).  Shapes are ragged on purpose: token counts around the
64- and 128-token tile sizes, a short last block, head counts that leave trailing CTAs.
"""
import ctypes

import numpy as np
import pytest

import synth
from parity_util import to_dev

pytestmark = pytest.mark.gpu

EPS = 1e-6
BAND = 8192          # bytes of guard on each side of a buffer (a multiple of 256: carved buffers stay aligned)
PATTERN = 0xA5


@pytest.fixture(scope="module")
def la():
    import torch

    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2509_24695_b200 as la

    la.load_library()
    return la


class Pool:
    """Carves guarded buffers out of torch byte tensors and checks the guards."""

    def __init__(self):
        self.items = []

    def take(self, shape, dtype):
        import torch

        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        pad = (-n) % 256
        raw = torch.full((BAND + n + pad + BAND,), PATTERN, dtype=torch.uint8, device="cuda")
        self.items.append((raw, n))
        return raw[BAND:BAND + n].view(dtype).view(shape)

    def check(self, what):
        import torch

        torch.cuda.synchronize()
        for i, (raw, n) in enumerate(self.items):
            front, back = raw[:BAND], raw[BAND + n:]
            assert bool((front == PATTERN).all()), f"{what}: bytes before buffer {i} ({n} bytes) were overwritten"
            assert bool((back == PATTERN).all()), f"{what}: bytes after buffer {i} ({n} bytes) were overwritten"


def tdtype(dtype):
    import torch

    return torch.bfloat16 if dtype == "bf16" else torch.float32


def gen(shape, seed, dtype):
    return tuple(to_dev(synth.gauss(shape, seed, t, dtype=dtype)) for t in (1, 2, 3))


RAGGED_N = [1, 63, 65, 127, 129, 1000]


@pytest.mark.parametrize("dtype,H,d", [("bf16", 3, 112), ("bf16", 20, 112), ("bf16", 5, 64), ("bf16", 8, 32), ("bf16", 2, 128),
                                       ("bf16", 3, 40), ("f32", 2, 112)])
def test_forward_state_apply_stay_inside_their_buffers(la, dtype, H, d):
    import torch

    for B, N in [(1, n) for n in RAGGED_N] + [(2, 321)]:
        pool = Pool()
        q, k, v = gen((B, N, H, d), 8000 + N + d, dtype)
        nws = la.workspace_bytes(B, H, d, N, la._dtype_code(q))
        ws = pool.take((nws,), torch.uint8)
        ws[:la.WORKSPACE_CTRL_BYTES] = 0
        o = pool.take((B, N, H, d), tdtype(dtype))
        st = pool.take((B, H, d + 1, d), torch.float32)
        la.linattn_forward(q, k, v, EPS, out=o, workspace=ws)
        pool.check(f"forward {dtype} B{B} N{N} H{H} d{d}")
        la.linattn_state(k, v, out=st, workspace=ws)
        pool.check(f"state {dtype} B{B} N{N} H{H} d{d}")
        la.linattn_apply(q, st, EPS, out=o, workspace=ws)
        pool.check(f"apply {dtype} B{B} N{N} H{H} d{d}")
        assert torch.isfinite(o.float()).all() and la.workspace_status(ws) == 0
        if d % 2 == 0:
            cos = torch.rand((N, d // 2), device="cuda") * 2 - 1
            table = la.rope_pack(cos, torch.sqrt(1 - cos * cos))
            nb = ctypes.c_size_t()
            la._check(la.load_library().linattn_rope_workspace_bytes(ctypes.byref(la._Desc(B, H, d, la._dtype_code(q), 0, 0, 0)),
                                                                     N, ctypes.byref(nb)), "linattn_rope_workspace_bytes")
            wsr = pool.take((nb.value,), torch.uint8)
            wsr[:la.WORKSPACE_CTRL_BYTES] = 0
            la.linattn_forward_rope(q, k, v, table, EPS, out=o, workspace=wsr)
            pool.check(f"rotary forward {dtype} B{B} N{N} H{H} d{d}")
            assert torch.isfinite(o.float()).all() and la.workspace_status(wsr) == 0


@pytest.mark.parametrize("dtype,H,d", [("bf16", 3, 112), ("bf16", 20, 112), ("bf16", 6, 64), ("f32", 2, 112), ("bf16", 3, 40),
                                       ("bf16", 5, 128)])
def test_block_cache_calls_stay_inside_their_buffers(la, dtype, H, d):
    """step, peek, absorb, prefill (block by block and all blocks together), and the rotary forms, on blocks whose
    last one is short, with the cache's state and workspace between guard bands."""
    import torch

    B, T_b, M = 2, 129, 3
    N = T_b * M
    for joint in (0, M):
        pool = Pool()
        sbytes, wbytes = la.BlockLinCache.sizes(B, H, d, tdtype(dtype), T_b, prefill_blocks=joint)
        state = pool.take((B, H, d + 1, d), torch.float32)
        ws = pool.take((wbytes,), torch.uint8)
        assert sbytes == state.numel() * 4
        cache = la.BlockLinCache(B, H, d, tdtype(dtype), "cuda", max_T_b=T_b, eps=EPS, prefill_blocks=joint, state=state,
                                 workspace=ws)
        q, k, v = gen((B, N, H, d), 8100 + d, dtype)
        o_full = pool.take((B, N, H, d), tdtype(dtype))
        cos = torch.rand((N, d // 2), device="cuda") * 2 - 1
        table = la.rope_pack(cos, torch.sqrt(1 - cos * cos))
        what = f"{dtype} H{H} d{d} joint{joint}"
        for T in (T_b, 65, 1):                                    # a full block, a short one, a single token
            blk = [x[:, :T].contiguous() for x in (q, k, v)]
            o = pool.take((B, T, H, d), tdtype(dtype))
            cache.step(*blk, out=o); pool.check("step " + what)
            cache.peek(*blk, out=o); pool.check("peek " + what)
            cache.step(None, blk[1], blk[2]); pool.check("absorb " + what)
            cache.step_rope(*blk, table[:T].contiguous(), out=o); pool.check("rotary step " + what)
            cache.peek_rope(*blk, table[:T].contiguous(), out=o); pool.check("rotary peek " + what)
            assert torch.isfinite(o.float()).all()
        cache.reset()
        # prefill over token ranges of the long tensors (blocks keep the long tensors' batch stride)
        cache2 = la.BlockLinCache(B, H, d, tdtype(dtype), "cuda", max_T_b=T_b, eps=EPS, prefill_blocks=joint, state=state,
                                  workspace=ws, strides=tuple(q.stride()[:3]))
        cache2.prefill(q, k, v, M, out=o_full); pool.check("prefill " + what)
        cache2.prefill_rope(q, k, v, table, M, out=o_full); pool.check("rotary prefill " + what)
        assert torch.isfinite(o_full.float()).all() and torch.isfinite(state).all()
        assert cache2.status() == 0
        cache.close(); cache2.close()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_tconv_calls_stay_inside_their_buffers(la, dtype):
    import torch

    for B, T, HW, D, T_b in ((2, 7, 37, 72, 3), (1, 3, 129, 40, 3), (2, 4, 9, 2240, 1), (1, 1, 11, 24, 1)):
        pool = Pool()
        x = to_dev(synth.gauss((B, T, HW, D), 8200 + HW, 1, dtype=dtype))
        w = to_dev(synth.gauss((3, D), 8201, 2, dtype="f32"))
        y = pool.take((B, T, HW, D), tdtype(dtype))
        frame = pool.take((B, HW, D), tdtype(dtype))
        what = f"tconv {dtype} B{B} T{T} HW{HW} D{D}"
        la.tconv_forward(x, w, out=y); pool.check("forward " + what)
        cache = la.TConvCache(B, HW, D, tdtype(dtype), "cuda", frame=frame)
        for t0 in range(0, T, T_b):
            blk = x[:, t0:t0 + T_b]
            cache.step(blk, w, out=y[:, t0:t0 + T_b], commit=False); pool.check("read-only step " + what)
            cache.step(blk, w, out=y[:, t0:t0 + T_b]); pool.check("step " + what)
        cache.absorb(x[:, :T_b]); pool.check("absorb " + what)
        if T % T_b == 0:
            cache.prefill(x, w, T // T_b, out=y); pool.check("prefill " + what)
        assert torch.isfinite(y.float()).all() and torch.isfinite(frame.float()).all()
