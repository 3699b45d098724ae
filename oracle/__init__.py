"""ctypes front end of the fp64 CPU oracle (``linattn_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Nothing under the product package may import this
module; it exists so tests, the smoke check and the benchmark's CPU legs can
compute what the paper's equations say, independently of the CUDA kernels.

Inputs are numpy arrays ``[B, N, H, d]`` (any strides with a contiguous last
axis) of dtype uint16 (bfloat16 bit patterns), float32 or float64.  Outputs
are float64.  State arrays are ``S[B,H,d,d]`` (key feature, value feature) and
``z[B,H,d]``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
SOURCE = os.path.join(_HERE, "linattn_oracle.c")
_LIB = os.path.join(_HERE, "liblinattn_oracle.so")
CFLAGS = ["-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC"]


def build(force: bool = False, source: str = SOURCE, out: str = _LIB) -> str:
    """Compile the oracle with gcc (fp contraction off so fp64 stays plain)."""
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(source):
        tmp = out + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", *CFLAGS, "-o", tmp, source, "-lm"])
        os.replace(tmp, out)
    return out


class _Shape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in ("B", "N", "H", "d", "stride_b", "stride_n", "stride_h")] + [
        ("dtype", ctypes.c_int32)
    ]


_DT = {np.dtype(np.uint16): 0, np.dtype(np.float32): 1, np.dtype(np.float64): 2}


def _bind(path: str):
    lib = ctypes.CDLL(path)
    vp, dp, sp = ctypes.c_void_p, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(_Shape)
    i64, f64 = ctypes.c_int64, ctypes.c_double
    lib.oracle_state.argtypes = [sp, vp, vp, dp, dp]
    lib.oracle_apply_rows.argtypes = [sp, vp, dp, dp, f64, ctypes.POINTER(i64), i64, dp]
    lib.oracle_linattn_forward.argtypes = [sp, vp, vp, vp, f64, dp]
    lib.oracle_quadratic.argtypes = [sp, vp, vp, vp, f64, i64, dp]
    lib.oracle_block_step.argtypes = [sp, vp, vp, vp, f64, dp, dp, dp]
    lib.oracle_block_masked.argtypes = [sp, vp, vp, vp, f64, i64, dp]
    lib.oracle_rope_forward.argtypes = [sp, vp, vp, vp, dp, dp, f64, dp]
    lib.oracle_rope_quadratic.argtypes = [sp, vp, vp, vp, dp, dp, f64, i64, dp]
    lib.oracle_rope_block_masked.argtypes = [sp, vp, vp, vp, dp, dp, f64, i64, dp]
    lib.oracle_rope_block_step.argtypes = [sp, vp, vp, vp, dp, dp, f64, dp, dp, dp]
    lib.oracle_cache_bytes.argtypes = [i64, i64, i64]
    lib.oracle_cache_bytes.restype = i64
    return lib


class Oracle:
    """One loaded oracle library (the default build, or a mutant built by a test)."""

    def __init__(self, path: str | None = None):
        self._lib = _bind(path or build())

    @staticmethod
    def _shape(*arrs):
        a0 = arrs[0]
        assert a0.ndim == 4, "tensors are [B, N, H, d]"
        for a in arrs:
            assert a.shape == a0.shape and a.dtype == a0.dtype
            assert a.strides == a0.strides, "q, k, v must share one memory layout"
            assert a.dtype in _DT, a.dtype
            assert a.strides[3] == a.itemsize, "last axis must be contiguous"
        B, N, H, d = a0.shape
        it = a0.itemsize
        sb, sn, sh = (a0.strides[0] // it, a0.strides[1] // it, a0.strides[2] // it)
        return _Shape(B, N, H, d, sb, sn, sh, _DT[a0.dtype])

    @staticmethod
    def _dp(a):
        assert a.dtype == np.float64 and a.flags.c_contiguous
        return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))

    def state(self, k, v):
        s = self._shape(k, v)
        S = np.empty((s.B, s.H, s.d, s.d)); z = np.empty((s.B, s.H, s.d))
        self._lib.oracle_state(ctypes.byref(s), k.ctypes.data, v.ctypes.data, self._dp(S), self._dp(z))
        return S, z

    def apply_rows(self, q, S, z, eps, rows):
        s = self._shape(q)
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        assert rows.size == 0 or (0 <= rows.min() and rows.max() < s.N)
        o = np.empty((s.B, rows.size, s.H, s.d))
        self._lib.oracle_apply_rows(ctypes.byref(s), q.ctypes.data, self._dp(S), self._dp(z), eps,
                                    rows.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), rows.size, self._dp(o))
        return o

    def forward(self, q, k, v, eps):
        s = self._shape(q, k, v)
        o = np.empty((s.B, s.N, s.H, s.d))
        self._lib.oracle_linattn_forward(ctypes.byref(s), q.ctypes.data, k.ctypes.data, v.ctypes.data, eps, self._dp(o))
        return o

    def quadratic(self, q, k, v, eps, T_b: int = 0):
        s = self._shape(q, k, v)
        o = np.empty((s.B, s.N, s.H, s.d))
        self._lib.oracle_quadratic(ctypes.byref(s), q.ctypes.data, k.ctypes.data, v.ctypes.data, eps, T_b, self._dp(o))
        return o

    def block_masked(self, q, k, v, eps, T_b: int):
        s = self._shape(q, k, v)
        o = np.empty((s.B, s.N, s.H, s.d))
        self._lib.oracle_block_masked(ctypes.byref(s), q.ctypes.data, k.ctypes.data, v.ctypes.data, eps, T_b, self._dp(o))
        return o

    def rope_forward(self, q, k, v, cos, sin, eps, quadratic: bool = False, T_b: int = 0):
        """Eq. 2 with rotary factors in the numerator only.  cos, sin: [N, d//2] (any float dtype; widened
        exactly to fp64), the rotation of feature pair (2p, 2p+1) of token n.  T_b > 0: block-causal
        (quadratic: masked brute force; else block by block with the running cache)."""
        s = self._shape(q, k, v)
        cs = np.ascontiguousarray(cos, dtype=np.float64)
        sn = np.ascontiguousarray(sin, dtype=np.float64)
        assert cs.shape == sn.shape == (s.N, s.d // 2)
        o = np.empty((s.B, s.N, s.H, s.d))
        args = (ctypes.byref(s), q.ctypes.data, k.ctypes.data, v.ctypes.data, self._dp(cs), self._dp(sn), eps)
        if quadratic:
            self._lib.oracle_rope_quadratic(*args, T_b, self._dp(o))
        elif T_b > 0:
            self._lib.oracle_rope_block_masked(*args, T_b, self._dp(o))
        else:
            self._lib.oracle_rope_forward(*args, self._dp(o))
        return o

    def new_cache(self, B, H, d):
        """An empty cache: the running (sum S, sum phi(K)^T) pair, all zeros."""
        return np.zeros((B, H, d, d)), np.zeros((B, H, d))

    def block_step(self, cache, q, k, v, eps, want_o: bool = True):
        """cache += state(block); returns apply(q_blk, cache) (or None)."""
        S, z = cache
        s = self._shape(q, k, v)
        o = np.empty((s.B, s.N, s.H, s.d)) if want_o else None
        self._lib.oracle_block_step(ctypes.byref(s), q.ctypes.data, k.ctypes.data, v.ctypes.data, eps,
                                    self._dp(S), self._dp(z), self._dp(o) if want_o else None)
        return o

    def rope_block_step(self, cache, q, k, v, cos_blk, sin_blk, eps, want_o: bool = True):
        """``block_step`` with rotary factors: cache += (RoPE(phi(k))^T v, phi(k)) of the block, then the block's
        queries read it.  cos_blk, sin_blk: [T_b, d//2], the table rows of the block's tokens."""
        S, z = cache
        s = self._shape(q, k, v)
        cs = np.ascontiguousarray(cos_blk, dtype=np.float64)
        sn = np.ascontiguousarray(sin_blk, dtype=np.float64)
        assert cs.shape == sn.shape == (s.N, s.d // 2)
        o = np.empty((s.B, s.N, s.H, s.d)) if want_o else None
        self._lib.oracle_rope_block_step(ctypes.byref(s), q.ctypes.data, k.ctypes.data, v.ctypes.data, self._dp(cs),
                                         self._dp(sn), eps, self._dp(S), self._dp(z), self._dp(o) if want_o else None)
        return o

    def cache_bytes(self, B, H, d) -> int:
        return int(self._lib.oracle_cache_bytes(B, H, d))


_default = None


def default() -> Oracle:
    global _default
    if _default is None:
        _default = Oracle()
    return _default
