"""ReLU linear attention for B200 (sm_100a): thin Python binding of the C-ABI library.

Every function here only marshals arguments (device pointers, sizes, strides, the
current CUDA stream) into the ``extern "C"`` entry points declared in
``include/linattn.h``; all arithmetic runs in the library's CUDA kernels.  PyTorch is
used for device memory and streams only.  There is no CPU fallback: if the shared
library cannot be loaded or built, or a call returns an error status, a
``LinAttnError`` is raised.

Tensors are ``[B, N, H, d]`` torch CUDA tensors (bfloat16 or float32) whose last axis
is contiguous.  A state is a float32 tensor ``[B, H, d+1, d]``: rows ``0..d-1`` hold
``S`` transposed (``state[b,h,j,i] = S[i,j]``), row ``d`` holds ``z``.
"""
from __future__ import annotations

import ctypes
import os

__all__ = [
    "LinAttnError", "library_path", "load_library", "state_bytes", "workspace_bytes", "new_workspace",
    "linattn_forward", "linattn_forward_rope", "rope_pack", "new_rope_workspace", "linattn_state", "linattn_apply", "linattn_state_static_scratch", "static_scratch_status", "split_state", "BlockLinCache", "workspace_status", "HostForward", "kernel_launches",
    "tconv_forward", "TConvCache",
]

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "liblinattn.so")

LINATTN_BF16, LINATTN_F32 = 0, 1
WORKSPACE_CTRL_BYTES = 4096


class LinAttnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib.linattn_status_string(status).decode() if _lib is not None else "library not loaded"
        super().__init__(f"{where}: {msg} (status {status})")


class _Desc(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("d", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("stride_b", ctypes.c_int64), ("stride_n", ctypes.c_int64), ("stride_h", ctypes.c_int64)]


class _ConvDesc(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("HW", ctypes.c_int32), ("D", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("stride_b", ctypes.c_int64), ("stride_b_y", ctypes.c_int64)]


_lib = None


def library_path() -> str:
    return _LIB_PATH


def load_library(path: str | None = None):
    """Load ``liblinattn.so`` (building it in-tree with nvcc first if it is absent)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or _LIB_PATH
    if not os.path.exists(p):
        from . import build as _build  # raises if nvcc fails: no fallback exists

        p = _build.build()
    lib = ctypes.CDLL(p)
    vp, i64, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t
    dp = ctypes.POINTER(_Desc)
    szp = ctypes.POINTER(sz)
    f32 = ctypes.c_float
    sig = {
        "linattn_status_string": ([ctypes.c_int], ctypes.c_char_p),
        "linattn_state_bytes": ([dp, szp], ctypes.c_int),
        "linattn_workspace_bytes": ([dp, i64, szp], ctypes.c_int),
        "linattn_workspace_init": ([vp, sz, vp], ctypes.c_int),
        "linattn_workspace_status": ([vp, vp, ctypes.POINTER(ctypes.c_int)], ctypes.c_int),
        "linattn_forward": ([dp, i64, vp, vp, vp, vp, f32, vp, sz, vp], ctypes.c_int),
        "linattn_rope_workspace_bytes": ([dp, i64, szp], ctypes.c_int),
        "linattn_rope_table_bytes": ([i64, ctypes.c_int32, szp], ctypes.c_int),
        "linattn_rope_pack": ([i64, ctypes.c_int32, vp, vp, vp, vp], ctypes.c_int),
        "linattn_forward_rope": ([dp, i64, vp, vp, vp, vp, f32, vp, vp, sz, vp], ctypes.c_int),
        "linattn_state": ([dp, i64, vp, vp, vp, vp, sz, vp], ctypes.c_int),
        "linattn_apply": ([dp, i64, vp, vp, vp, f32, vp, sz, vp], ctypes.c_int),
        "linattn_state_static_scratch": ([dp, i64, vp, vp, vp, vp], ctypes.c_int),
        "linattn_forward_host_bytes": ([dp, i64, szp], ctypes.c_int),
        "linattn_forward_host": ([dp, i64, vp, vp, vp, vp, f32, vp, sz, vp], ctypes.c_int),
        "linattn_kernel_launches": ([], ctypes.c_uint64),
        "blocklin_cache_bytes": ([dp, i64, szp, szp], ctypes.c_int),
        "blocklin_cache_init": ([ctypes.POINTER(vp), dp, f32, vp, sz, vp, sz, vp], ctypes.c_int),
        "blocklin_cache_reset": ([vp, vp], ctypes.c_int),
        "blocklin_step": ([vp, i64, vp, vp, vp, vp, vp], ctypes.c_int),
        "blocklin_peek": ([vp, i64, vp, vp, vp, vp, vp], ctypes.c_int),
        "blocklin_step_rope": ([vp, i64, vp, vp, vp, vp, vp, vp], ctypes.c_int),
        "blocklin_peek_rope": ([vp, i64, vp, vp, vp, vp, vp, vp], ctypes.c_int),
        "blocklin_prefill_rope": ([vp, i64, i64, vp, vp, vp, vp, vp, vp], ctypes.c_int),
        "blocklin_cache_status": ([vp, vp, ctypes.POINTER(ctypes.c_int)], ctypes.c_int),
        "linattn_static_scratch_status": ([vp, ctypes.POINTER(ctypes.c_int)], ctypes.c_int),
        "blocklin_prefill": ([vp, i64, i64, vp, vp, vp, vp, vp], ctypes.c_int),
        "blocklin_shard_state": ([vp, i64, vp, vp, vp, ctypes.c_int, vp], ctypes.c_int),
        "blocklin_shard_commit": ([vp, vp, i64, vp], ctypes.c_int),
        "blocklin_prefill_workspace_bytes": ([dp, i64, i64, szp], ctypes.c_int),
        "blocklin_cache_joint_prefill": ([vp, ctypes.c_int], ctypes.c_int),
        "blocklin_cache_info": ([vp, ctypes.POINTER(i64), ctypes.POINTER(i64), szp], ctypes.c_int),
        "blocklin_cache_destroy": ([vp], ctypes.c_int),
        "tconv_cache_bytes": ([ctypes.POINTER(_ConvDesc), szp], ctypes.c_int),
        "tconv_cache_reset": ([ctypes.POINTER(_ConvDesc), vp, vp], ctypes.c_int),
        "tconv_forward": ([ctypes.POINTER(_ConvDesc), i64, vp, vp, vp, vp], ctypes.c_int),
        "tconv_block_step": ([ctypes.POINTER(_ConvDesc), i64, vp, vp, vp, vp, ctypes.c_int, vp], ctypes.c_int),
        "tconv_prefill": ([ctypes.POINTER(_ConvDesc), i64, i64, vp, vp, vp, vp, vp], ctypes.c_int),
    }
    for name, (argtypes, restype) in sig.items():
        fn = getattr(lib, name)
        fn.argtypes, fn.restype = argtypes, restype
    if path is None:
        _lib = lib
    return lib


def _check(status: int, where: str):
    if status != 0:
        raise LinAttnError(status, where)


def _torch():
    import torch

    return torch


def _dtype_code(t) -> int:
    torch = _torch()
    if t.dtype == torch.bfloat16:
        return LINATTN_BF16
    if t.dtype == torch.float32:
        return LINATTN_F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _desc_of(t, *same) -> _Desc:
    """Descriptor for a [B, N, H, d] tensor; every tensor in `same` must share its layout."""
    if t.dim() != 4 or t.stride(3) != 1 or not t.is_cuda:
        raise ValueError("expected a CUDA tensor [B, N, H, d] with a contiguous last axis")
    for o in same:
        if o.shape != t.shape or o.stride() != t.stride() or o.dtype != t.dtype or o.device != t.device:
            raise ValueError("q, k, v, o must share shape, strides, dtype and device")
    B, N, H, d = t.shape
    return _Desc(B, H, d, _dtype_code(t), t.stride(0), t.stride(1), t.stride(2))


def _stream(t) -> int:
    return _torch().cuda.current_stream(t.device).cuda_stream


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else None


def state_bytes(B: int, H: int, d: int) -> int:
    lib = load_library()
    out = ctypes.c_size_t()
    _check(lib.linattn_state_bytes(ctypes.byref(_Desc(B, H, d, 0, 0, 0, 0)), ctypes.byref(out)), "linattn_state_bytes")
    return out.value


def workspace_bytes(B: int, H: int, d: int, N: int, dtype_code: int = LINATTN_BF16) -> int:
    lib = load_library()
    out = ctypes.c_size_t()
    _check(lib.linattn_workspace_bytes(ctypes.byref(_Desc(B, H, d, dtype_code, 0, 0, 0)), N, ctypes.byref(out)),
           "linattn_workspace_bytes")
    return out.value


def new_workspace(like, N: int | None = None):
    """Allocate (with torch) and initialise a workspace fit for tensors shaped like `like`."""
    torch = _torch()
    lib = load_library()
    B, n, H, d = like.shape
    nbytes = workspace_bytes(B, H, d, n if N is None else N, _dtype_code(like))
    ws = torch.empty(nbytes, dtype=torch.uint8, device=like.device)
    _check(lib.linattn_workspace_init(_ptr(ws), nbytes, _stream(like)), "linattn_workspace_init")
    return ws


def workspace_status(ws) -> int:
    lib = load_library()
    st = ctypes.c_int(0)
    _check(lib.linattn_workspace_status(_ptr(ws), _stream(ws), ctypes.byref(st)), "linattn_workspace_status")
    return st.value


def linattn_forward(q, k, v, eps: float = 1e-6, out=None, workspace=None):
    """Bidirectional ReLU linear attention (Eq. 2): returns O with the layout of q."""
    torch = _torch()
    lib = load_library()
    o = torch.empty_like(q) if out is None else out
    desc = _desc_of(q, k, v, o)
    ws = new_workspace(q) if workspace is None else workspace
    _check(lib.linattn_forward(ctypes.byref(desc), q.shape[1], _ptr(q), _ptr(k), _ptr(v), _ptr(o), eps,
                               _ptr(ws), ws.numel(), _stream(q)), "linattn_forward")
    return o


def rope_pack(rope_cos, rope_sin):
    """Packed rotary table for ``linattn_forward_rope``: float32 CUDA tensors [N, d//2] of the pair rotations'
    cosines and sines -> one [N, d//2, 2] float16 tensor (cos, sin), rounded to nearest by the library."""
    torch = _torch()
    lib = load_library()
    if rope_cos.shape != rope_sin.shape or rope_cos.dim() != 2 or rope_cos.dtype != torch.float32 or \
            rope_sin.dtype != torch.float32 or not rope_cos.is_contiguous() or not rope_sin.is_contiguous():
        raise ValueError("rope_cos and rope_sin must be contiguous float32 [N, d//2] tensors")
    N, half = rope_cos.shape
    table = torch.empty((N, half, 2), dtype=torch.float16, device=rope_cos.device)
    _check(lib.linattn_rope_pack(N, 2 * half, _ptr(rope_cos), _ptr(rope_sin), _ptr(table), _stream(rope_cos)),
           "linattn_rope_pack")
    return table


def new_rope_workspace(like):
    """Allocate (with torch) and initialise a workspace for ``linattn_forward_rope`` on tensors shaped like `like`."""
    torch = _torch()
    lib = load_library()
    B, N, H, d = like.shape
    nb = ctypes.c_size_t()
    _check(lib.linattn_rope_workspace_bytes(ctypes.byref(_Desc(B, H, d, _dtype_code(like), 0, 0, 0)), N, ctypes.byref(nb)),
           "linattn_rope_workspace_bytes")
    ws = torch.empty(nb.value, dtype=torch.uint8, device=like.device)
    _check(lib.linattn_workspace_init(_ptr(ws), nb.value, _stream(like)), "linattn_workspace_init")
    return ws


def linattn_forward_rope(q, k, v, rope_table, eps: float = 1e-6, out=None, workspace=None):
    """Eq. 2 with its rotary factors (rotation after the ReLU, numerator only).  rope_table: the float16
    [N, d//2, 2] (cos, sin) table of ``rope_pack``: the rotation of feature pair (2p, 2p+1) of token n."""
    torch = _torch()
    lib = load_library()
    o = torch.empty_like(q) if out is None else out
    desc = _desc_of(q, k, v, o)
    B, N, H, d = q.shape
    if tuple(rope_table.shape) != (N, d // 2, 2) or rope_table.dtype != torch.float16 or \
            not rope_table.is_contiguous() or rope_table.device != q.device:
        raise ValueError("rope_table must be a contiguous float16 [N, d//2, 2] tensor on the device of q")
    if workspace is None:
        workspace = new_rope_workspace(q)
    _check(lib.linattn_forward_rope(ctypes.byref(desc), N, _ptr(q), _ptr(k), _ptr(v), _ptr(o), eps, _ptr(rope_table),
                                    _ptr(workspace), workspace.numel(), _stream(q)), "linattn_forward_rope")
    return o


def kernel_launches() -> int:
    """CUDA kernels launched by the library in this process so far."""
    return int(load_library().linattn_kernel_launches())


class HostForward:
    """Bidirectional forward over HOST tensors (pinned CPU torch tensors, dense [B, N, H, d]).

    Owns a device staging area (allocated once with torch); each call enqueues host-to-device copies
    of Q, K, V, the forward, and the device-to-host copy of O on the current stream.
    """

    def __init__(self, B: int, N: int, H: int, d: int, dtype, device="cuda"):
        torch = _torch()
        self._lib = load_library()
        code = LINATTN_BF16 if dtype == torch.bfloat16 else LINATTN_F32
        self._desc = _Desc(B, H, d, code, 0, 0, 0)
        self.shape, self.dtype, self.N = (B, N, H, d), dtype, N
        nb = ctypes.c_size_t()
        _check(self._lib.linattn_forward_host_bytes(ctypes.byref(self._desc), N, ctypes.byref(nb)),
               "linattn_forward_host_bytes")
        self.staging = torch.empty(nb.value, dtype=torch.uint8, device=device)
        _check(self._lib.linattn_workspace_init(_ptr(self.staging), nb.value, _stream(self.staging)),
               "linattn_workspace_init")
        itemsize = 2 if code == LINATTN_BF16 else 4
        self.h2d_bytes = 3 * B * N * H * d * itemsize
        self.d2h_bytes = B * N * H * d * itemsize

    def __call__(self, q_host, k_host, v_host, o_host, eps: float = 1e-6):
        for t in (q_host, k_host, v_host, o_host):
            if t.is_cuda or tuple(t.shape) != self.shape or t.dtype != self.dtype or not t.is_contiguous():
                raise ValueError("host tensors must be dense CPU [B, N, H, d] tensors of the configured dtype")
        _check(self._lib.linattn_forward_host(ctypes.byref(self._desc), self.N, _ptr(q_host), _ptr(k_host),
                                              _ptr(v_host), _ptr(o_host), eps, _ptr(self.staging),
                                              self.staging.numel(), _stream(self.staging)), "linattn_forward_host")
        return o_host


def linattn_state(k, v, out=None, workspace=None):
    """State of Eq. 2 / Eq. 3: float32 [B, H, d+1, d] (S transposed, then z)."""
    torch = _torch()
    lib = load_library()
    desc = _desc_of(k, v)
    B, N, H, d = k.shape
    st = torch.empty((B, H, d + 1, d), dtype=torch.float32, device=k.device) if out is None else out
    ws = new_workspace(k) if workspace is None else workspace
    _check(lib.linattn_state(ctypes.byref(desc), N, _ptr(k), _ptr(v), _ptr(st), _ptr(ws), ws.numel(), _stream(k)),
           "linattn_state")
    return st


STATIC_SCRATCH_BYTES = 16 << 20


def linattn_state_static_scratch(k, v, out):
    """``linattn_state`` without a workspace: for callers that must not allocate device memory.

    The split-N scratch is an array built into the library (``STATIC_SCRATCH_BYTES``, shared by all
    calls on a device), so this wrapper allocates nothing either: ``out`` (float32 ``[B, H, d+1, d]``)
    is required.  Problems whose scratch does not fit raise ``LinAttnError`` with status -8.  Calls
    on one device must not overlap on the GPU; make the first call outside stream capture.
    """
    torch = _torch()
    lib = load_library()
    desc = _desc_of(k, v)
    B, N, H, d = k.shape
    if tuple(out.shape) != (B, H, d + 1, d) or out.dtype != torch.float32 or not out.is_contiguous():
        raise ValueError("out must be a contiguous float32 [B, H, d+1, d] tensor")
    _check(lib.linattn_state_static_scratch(ctypes.byref(desc), N, _ptr(k), _ptr(v), _ptr(out), _stream(k)),
           "linattn_state_static_scratch")
    return out


def static_scratch_status(device=None) -> int:
    """Device-side status (0 or -6) of the last ``linattn_state_static_scratch`` call on the current device."""
    torch = _torch()
    lib = load_library()
    st = ctypes.c_int(0)
    _check(lib.linattn_static_scratch_status(torch.cuda.current_stream(device).cuda_stream, ctypes.byref(st)),
           "linattn_static_scratch_status")
    return st.value


def linattn_apply(q, state, eps: float = 1e-6, out=None, workspace=None):
    """Apply half of Eq. 2 for a given state."""
    torch = _torch()
    lib = load_library()
    o = torch.empty_like(q) if out is None else out
    desc = _desc_of(q, o)
    B, N, H, d = q.shape
    if tuple(state.shape) != (B, H, d + 1, d) or state.dtype != torch.float32 or not state.is_contiguous():
        raise ValueError("state must be a contiguous float32 [B, H, d+1, d] tensor")
    ws = new_workspace(q, 0) if workspace is None else workspace
    _check(lib.linattn_apply(ctypes.byref(desc), N, _ptr(q), _ptr(state), _ptr(o), eps, _ptr(ws), ws.numel(),
                             _stream(q)), "linattn_apply")
    return o


def split_state(state):
    """Views (S [B,H,d,d] indexed [key feature, value feature], z [B,H,d]) of a state tensor."""
    d = state.shape[-1]
    return state[..., :d, :].transpose(-1, -2), state[..., d, :]


class BlockLinCache:
    """Constant-memory cache of the block-causal form (Eq. 3, Algorithm 1's cache).

    Owns (through torch) the fp32 state ``[B, H, d+1, d]`` and a scratch workspace; the
    C handle only borrows their device pointers.  ``state`` is plain memory: cloning it
    checkpoints the stream, copying into it restores one.
    """

    def __init__(self, B: int, H: int, d: int, dtype, device, max_T_b: int, eps: float = 1e-6,
                 strides: tuple[int, int, int] = (0, 0, 0), prefill_blocks: int = 0, state=None, workspace=None):
        """state / workspace: caller-provided device tensors (a float32 ``[B, H, d+1, d]`` tensor and a uint8 tensor
        of at least ``workspace_bytes_needed`` bytes, both 16-byte aligned) for callers that manage their own
        pools; by default both are allocated here with torch."""
        torch = _torch()
        self._lib = load_library()
        code = LINATTN_BF16 if dtype == torch.bfloat16 else LINATTN_F32 if dtype == torch.float32 else None
        if code is None:
            raise TypeError(f"unsupported dtype {dtype}")
        self._desc = _Desc(B, H, d, code, *strides)
        state_bytes_, nbytes = self.sizes(B, H, d, dtype, max_T_b, prefill_blocks, strides)
        if state is None:
            state = torch.empty((B, H, d + 1, d), dtype=torch.float32, device=device)
        elif tuple(state.shape) != (B, H, d + 1, d) or state.dtype != torch.float32 or not state.is_contiguous():
            raise ValueError("state must be a contiguous float32 [B, H, d+1, d] tensor")
        self.state = state
        assert self.state.numel() * 4 == state_bytes_
        self.workspace_bytes_needed = nbytes
        if workspace is None:
            workspace = torch.empty(nbytes, dtype=torch.uint8, device=device)
        elif workspace.dtype != torch.uint8 or workspace.numel() < nbytes or not workspace.is_contiguous():
            raise ValueError(f"workspace must be a contiguous uint8 tensor of at least {nbytes} bytes")
        else:
            nbytes = workspace.numel()
        self.workspace = workspace
        self.max_T_b, self.eps = max_T_b, eps
        self._handle = ctypes.c_void_p()
        _check(self._lib.blocklin_cache_init(ctypes.byref(self._handle), ctypes.byref(self._desc), eps,
                                             _ptr(self.state), state_bytes_, _ptr(self.workspace), nbytes,
                                             _stream(self.state)), "blocklin_cache_init")
        if prefill_blocks > 1:
            _check(self._lib.blocklin_cache_joint_prefill(self._handle, 1), "blocklin_cache_joint_prefill")

    @staticmethod
    def sizes(B: int, H: int, d: int, dtype, max_T_b: int, prefill_blocks: int = 0, strides=(0, 0, 0)) -> tuple[int, int]:
        """(state bytes, workspace bytes) a cache of this shape needs; prefill_blocks > 1: room for ``prefill`` to
        take that many blocks of max_T_b tokens together."""
        torch = _torch()
        lib = load_library()
        desc = _Desc(B, H, d, LINATTN_BF16 if dtype == torch.bfloat16 else LINATTN_F32, *strides)
        sb, wb = ctypes.c_size_t(), ctypes.c_size_t()
        _check(lib.blocklin_cache_bytes(ctypes.byref(desc), max_T_b, ctypes.byref(sb), ctypes.byref(wb)), "blocklin_cache_bytes")
        nbytes = wb.value
        if prefill_blocks > 1:
            pb = ctypes.c_size_t()
            _check(lib.blocklin_prefill_workspace_bytes(ctypes.byref(desc), prefill_blocks, max_T_b, ctypes.byref(pb)),
                   "blocklin_prefill_workspace_bytes")
            nbytes = max(nbytes, pb.value)
        return sb.value, nbytes

    def reset(self):
        _check(self._lib.blocklin_cache_reset(self._handle, _stream(self.state)), "blocklin_cache_reset")

    def step(self, q, k, v, out=None):
        """cache += state(block); returns the block's output (None when q is None)."""
        torch = _torch()
        o = None
        if q is not None:
            o = torch.empty_like(q) if out is None else out
            _desc_of(q, k, v, o)
        else:
            _desc_of(k, v)
        self._check_layout(k)
        _check(self._lib.blocklin_step(self._handle, k.shape[1], _ptr(q), _ptr(k), _ptr(v), _ptr(o), _stream(k)),
               "blocklin_step")
        return o

    def _rope_args(self, q, k, v, table, out, rows):
        torch = _torch()
        o = None
        if q is not None:
            o = torch.empty_like(q) if out is None else out
            _desc_of(q, k, v, o)
        else:
            _desc_of(k, v)
        self._check_layout(k)
        d = k.shape[3]
        if tuple(table.shape) != (rows, d // 2, 2) or table.dtype != torch.float16 or not table.is_contiguous() \
                or table.device != k.device:
            raise ValueError("the rotary table must be a contiguous float16 [tokens, d//2, 2] tensor on the blocks' device")
        return o

    def step_rope(self, q, k, v, rope_table_blk, out=None):
        """``step`` with rotary factors; rope_table_blk: float16 [T_b, d//2, 2] rows of the block's tokens
        (a contiguous slice of the stream's ``rope_pack`` table).  q may be None: absorb only."""
        o = self._rope_args(q, k, v, rope_table_blk, out, k.shape[1])
        _check(self._lib.blocklin_step_rope(self._handle, k.shape[1], _ptr(q), _ptr(k), _ptr(v), _ptr(o),
                                            _ptr(rope_table_blk), _stream(k)), "blocklin_step_rope")
        return o

    def peek_rope(self, q, k, v, rope_table_blk, out=None):
        """``peek`` with rotary factors: the block against the rotary cache plus itself, nothing committed."""
        if q is None:
            raise ValueError("peek_rope needs queries")
        o = self._rope_args(q, k, v, rope_table_blk, out, k.shape[1])
        _check(self._lib.blocklin_peek_rope(self._handle, k.shape[1], _ptr(q), _ptr(k), _ptr(v), _ptr(o),
                                            _ptr(rope_table_blk), _stream(k)), "blocklin_peek_rope")
        return o

    def prefill_rope(self, q, k, v, rope_table, n_blocks: int, out=None):
        """n_blocks equal blocks with rotary factors in one call; rope_table: the rows of all their tokens."""
        N = k.shape[1]
        if n_blocks <= 0 or N % n_blocks:
            raise ValueError("token count must be n_blocks * T_b")
        o = self._rope_args(q, k, v, rope_table, out, N)
        _check(self._lib.blocklin_prefill_rope(self._handle, n_blocks, N // n_blocks, _ptr(q), _ptr(k), _ptr(v), _ptr(o),
                                               _ptr(rope_table), _stream(k)), "blocklin_prefill_rope")
        return o

    def status(self) -> int:
        """Synchronises the current stream; 0, or -6 if a bounded device-side wait of one of this cache's
        launches ran out (``reset`` clears it)."""
        st = ctypes.c_int(0)
        _check(self._lib.blocklin_cache_status(self._handle, _stream(self.state), ctypes.byref(st)),
               "blocklin_cache_status")
        return st.value

    def peek(self, q, k, v, out=None):
        """Output of the block against cache + state(block) without committing (Algorithm 1's denoising steps)."""
        torch = _torch()
        o = torch.empty_like(q) if out is None else out
        _desc_of(q, k, v, o)
        self._check_layout(k)
        _check(self._lib.blocklin_peek(self._handle, k.shape[1], _ptr(q), _ptr(k), _ptr(v), _ptr(o), _stream(k)),
               "blocklin_peek")
        return o

    def prefill(self, q, k, v, n_blocks: int, out=None):
        """n_blocks equal blocks in one call over [B, n_blocks*T_b, H, d] tensors."""
        torch = _torch()
        N = k.shape[1]
        if n_blocks <= 0 or N % n_blocks:
            raise ValueError("token count must be n_blocks * T_b")
        o = None
        if q is not None:
            o = torch.empty_like(q) if out is None else out
            _desc_of(q, k, v, o)
        else:
            _desc_of(k, v)
        self._check_layout(k)
        _check(self._lib.blocklin_prefill(self._handle, n_blocks, N // n_blocks, _ptr(q), _ptr(k), _ptr(v), _ptr(o),
                                          _stream(k)), "blocklin_prefill")
        return o

    def _check_layout(self, t):
        """The cache's descriptor fixes (B, H, d, dtype, strides); a block must match it."""
        dsc = self._desc
        if (t.shape[0], t.shape[2], t.shape[3]) != (dsc.B, dsc.H, dsc.d) or _dtype_code(t) != dsc.dtype:
            raise ValueError("block does not match the cache's (B, H, d, dtype)")
        want = (dsc.stride_b, dsc.stride_n, dsc.stride_h)
        if want == (0, 0, 0):
            if not t.is_contiguous():
                raise ValueError("this cache was created for dense [B, T_b, H, d] blocks")
        elif t.numel() and tuple(t.stride()[:3]) != want:
            raise ValueError(f"block strides {tuple(t.stride()[:3])} differ from the cache's {want}")

    def info(self) -> dict:
        b, t, s = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_size_t()
        _check(self._lib.blocklin_cache_info(self._handle, ctypes.byref(b), ctypes.byref(t), ctypes.byref(s)),
               "blocklin_cache_info")
        return {"blocks_seen": b.value, "tokens_seen": t.value, "state_bytes": s.value}

    def close(self):
        if self._handle:
            self._lib.blocklin_cache_destroy(self._handle)
            self._handle = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ---- temporal convolution of the Mix-FFN (tconv.h) ----

def _conv_desc_of(x, y=None) -> _ConvDesc:
    """Descriptor for x[B, T, HW, D] (and y): frames, positions and channels dense, any batch stride."""
    B, T, HW, D = x.shape if x.dim() == 4 else (0, 0, 0, 0)
    strides = []
    for t in (x, y):
        if t is None:
            strides.append(0)
            continue
        if t.dim() != 4 or not t.is_cuda or t.shape != x.shape or t.dtype != x.dtype or t.device != x.device:
            raise ValueError("expected CUDA tensors [B, T, HW, D] of one shape, dtype and device")
        if T > 0 and (t.stride(3) != 1 or t.stride(2) != D or (T > 1 and t.stride(1) != HW * D)):
            raise ValueError("frames, positions and channels must be dense")
        strides.append(t.stride(0) if B > 1 and T > 0 else 0)
    return _ConvDesc(B, HW, D, _dtype_code(x), strides[0], strides[1])


def _check_taps(w, D):
    torch = _torch()
    if w.dtype != torch.float32 or tuple(w.shape) != (3, D) or not w.is_contiguous() or not w.is_cuda:
        raise ValueError("taps must be a contiguous CUDA float32 tensor [3, D]")


def tconv_forward(x, w, out=None):
    """Bidirectional temporal convolution with shortcut over x[B, T, HW, D]; taps w[3, D] float32."""
    y = _torch().empty_like(x) if out is None else out
    desc = _conv_desc_of(x, y)
    _check_taps(w, x.shape[3])
    _check(load_library().tconv_forward(ctypes.byref(desc), x.shape[1], _ptr(x), _ptr(w), _ptr(y), _stream(x)),
           "tconv_forward")
    return y


class TConvCache:
    """The conv cache of the block-causal Mix-FFN: the last frame of the previous block, [B, HW, D]."""

    def __init__(self, B: int, HW: int, D: int, dtype, device, frame=None):
        torch = _torch()
        self._lib = load_library()
        if frame is not None and (tuple(frame.shape) != (B, HW, D) or frame.dtype != dtype or not frame.is_contiguous()):
            raise ValueError("frame must be a contiguous [B, HW, D] tensor of the cache's dtype")
        self.frame = torch.empty((B, HW, D), dtype=dtype, device=device) if frame is None else frame
        nbytes = ctypes.c_size_t()
        _check(self._lib.tconv_cache_bytes(ctypes.byref(self._desc(0)), ctypes.byref(nbytes)), "tconv_cache_bytes")
        assert nbytes.value == self.frame.numel() * self.frame.element_size()
        self.reset()

    def _desc(self, stride_b: int) -> _ConvDesc:
        B, HW, D = self.frame.shape
        return _ConvDesc(B, HW, D, _dtype_code(self.frame), stride_b, 0)

    def _desc_for(self, x, y=None) -> _ConvDesc:
        d = _conv_desc_of(x, y)
        if (d.B, d.HW, d.D, d.dtype) != (self.frame.shape[0], self.frame.shape[1], self.frame.shape[2],
                                         _dtype_code(self.frame)):
            raise ValueError("block does not match the cache's (B, HW, D, dtype)")
        return d

    def reset(self):
        _check(self._lib.tconv_cache_reset(ctypes.byref(self._desc(0)), _ptr(self.frame), _stream(self.frame)),
               "tconv_cache_reset")

    def step(self, x_blk, w, out=None, commit: bool = True):
        """One block x_blk[B, T_b, HW, D]; commit=False only reads the cache (a denoising step)."""
        y = _torch().empty_like(x_blk) if out is None else out
        d = self._desc_for(x_blk, y)
        _check_taps(w, d.D)
        _check(self._lib.tconv_block_step(ctypes.byref(d), x_blk.shape[1], _ptr(x_blk), _ptr(w), _ptr(self.frame),
                                          _ptr(y), int(commit), _stream(x_blk)), "tconv_block_step")
        return y

    def absorb(self, x_blk):
        """Take a block into the cache without computing its output."""
        d = self._desc_for(x_blk)
        _check(self._lib.tconv_block_step(ctypes.byref(d), x_blk.shape[1], _ptr(x_blk), None, _ptr(self.frame), None, 1,
                                          _stream(x_blk)), "tconv_block_step")

    def prefill(self, x, w, n_blocks: int, out=None):
        """n_blocks equal blocks of x[B, n_blocks*T_b, HW, D] in one launch."""
        T = x.shape[1]
        if n_blocks <= 0 or T % n_blocks:
            raise ValueError("frame count must be n_blocks * T_b")
        y = _torch().empty_like(x) if out is None else out
        d = self._desc_for(x, y)
        _check_taps(w, d.D)
        _check(self._lib.tconv_prefill(ctypes.byref(d), n_blocks, T // n_blocks, _ptr(x), _ptr(w), _ptr(self.frame),
                                       _ptr(y), _stream(x)), "tconv_prefill")
        return y
