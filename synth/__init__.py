"""Seeded synthetic inputs shaped like the paper's workloads.

Test and benchmark infrastructure only: this module holds none of the
attention arithmetic.  It is the one piece of code that both the CPU oracle's
callers and the CUDA path's callers use, so both sides start from identical
bit patterns.

Tensors are ``[B, N, H, d]`` (tokens ordered frame-major so that a block of
frames is a contiguous token range).  bfloat16 tensors are returned as numpy
``uint16`` arrays holding the raw bits.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "synth.c")
_LIB = os.path.join(_HERE, "libsynth.so")

Q_ID, K_ID, V_ID = 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the generator (gcc, a second or two). Returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u16p = ctypes.POINTER(ctypes.c_uint16)
        f32p = ctypes.POINTER(ctypes.c_float)
        i32p = ctypes.POINTER(ctypes.c_int32)
        i64, u64 = ctypes.c_int64, ctypes.c_uint64
        lib.synth_gauss_bf16.argtypes = [u16p, i64, u64, u64, i64, ctypes.c_double]
        lib.synth_gauss_f32.argtypes = [f32p, i64, u64, u64, i64, ctypes.c_double]
        lib.synth_smallint_bf16.argtypes = [u16p, i64, u64, u64, i64, ctypes.c_int32]
        lib.synth_index_i32.argtypes = [i32p, i64, u64, u64, i64, ctypes.c_int32]
        for f in (lib.synth_gauss_bf16, lib.synth_gauss_f32, lib.synth_smallint_bf16, lib.synth_index_i32):
            f.restype = None
        _lib = lib
    return _lib


def gauss(shape, seed: int, tensor_id: int, *, scale: float = 1.0, start: int = 0,
          dtype: str = "bf16", out: np.ndarray | None = None) -> np.ndarray:
    """N(0, scale^2) draws for flat indices ``start .. start+prod(shape)``.

    ``dtype='bf16'`` returns uint16 bit patterns (values rounded to nearest
    even from fp32); ``dtype='f32'`` returns float32.
    """
    lib = _load()
    count = int(np.prod(shape))
    if dtype == "bf16":
        a = out if out is not None else np.empty(shape, dtype=np.uint16)
        assert a.dtype == np.uint16 and a.size == count and a.flags.c_contiguous
        lib.synth_gauss_bf16(a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16)), count, seed, tensor_id, start, scale)
    elif dtype == "f32":
        a = out if out is not None else np.empty(shape, dtype=np.float32)
        assert a.dtype == np.float32 and a.size == count and a.flags.c_contiguous
        lib.synth_gauss_f32(a.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), count, seed, tensor_id, start, scale)
    else:
        raise ValueError(dtype)
    return a


def smallint(shape, seed: int, tensor_id: int, r: int = 2, *, start: int = 0) -> np.ndarray:
    """Integers drawn uniformly from {-r..r}, as bf16 bits (exact for r <= 128)."""
    lib = _load()
    a = np.empty(shape, dtype=np.uint16)
    lib.synth_smallint_bf16(a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16)), a.size, seed, tensor_id, start, r)
    return a


def index(shape, seed: int, tensor_id: int, n: int, *, start: int = 0) -> np.ndarray:
    """Uniform integers in [0, n) as int32."""
    lib = _load()
    a = np.empty(shape, dtype=np.int32)
    lib.synth_index_i32(a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), a.size, seed, tensor_id, start, n)
    return a


# ---- bf16 <-> float helpers for building structured inputs (bit manipulation only) ----

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 bits, nearest even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    u = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (u >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# ---- the five workload shapes ----

@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    d: int
    N: int          # tokens per call (bidirectional) or per whole stream (block form)
    seed: int
    scale: float    # multiplies the N(0,1) draws of Q, K and V before rounding
    T_b: int = 0    # tokens per block (0: bidirectional workload)
    n_blocks: int = 0
    eps: float = 1e-6

    @property
    def C(self) -> int:
        return self.H * self.d


TINY = Workload("tiny_bidir", B=1, H=4, d=32, N=3 * 8 * 8, seed=1001, scale=1.0)
P480 = Workload("480p_5s_bidir", B=1, H=20, d=112, N=21 * 30 * 52, seed=1002, scale=112 ** -0.5)
P720 = Workload("720p_5s_bidir", B=1, H=20, d=112, N=21 * 45 * 80, seed=1003, scale=1.0)
AR480 = Workload("480p_block_causal", B=1, H=20, d=112, N=7 * 4680, seed=1004, scale=1.0, T_b=3 * 30 * 52, n_blocks=7)
STREAM720 = Workload("720p_minute_stream", B=2, H=20, d=112, N=80 * 10800, seed=1005, scale=1.0, T_b=3 * 45 * 80, n_blocks=80)


def p720_sweep(d: int) -> Workload:
    """720p token count with another head dim at width ~2240: H = ceil(2240/d)."""
    H = -(-2240 // d)
    return Workload(f"720p_5s_bidir_d{d}", B=1, H=H, d=d, N=21 * 45 * 80, seed=1003 + d, scale=1.0)


def qkv(w: Workload, dtype: str = "bf16"):
    """Whole Q, K, V of a workload, each ``[B, N, H, d]``."""
    shape = (w.B, w.N, w.H, w.d)
    return tuple(gauss(shape, w.seed, t, scale=w.scale, dtype=dtype) for t in (Q_ID, K_ID, V_ID))


def qkv_block(w: Workload, blk: int, dtype: str = "bf16", n_tokens: int | None = None):
    """Q, K, V of block ``blk`` of a block-causal workload, each ``[B, T_b, H, d]``.

    Equals ``qkv(w)[..][:, blk*T_b:(blk+1)*T_b]`` without generating the stream.
    """
    T = w.T_b if n_tokens is None else n_tokens
    C = w.C
    outs = []
    for t in (Q_ID, K_ID, V_ID):
        a = np.empty((w.B, T, w.H, w.d), dtype=np.uint16 if dtype == "bf16" else np.float32)
        for b in range(w.B):
            gauss((T, w.H, w.d), w.seed, t, scale=w.scale, start=(b * w.N + blk * w.T_b) * C, dtype=dtype, out=a[b])
        outs.append(a)
    return tuple(outs)


def rope_axes(T: int, Hh: int, Ww: int, d: int, base: float = 10000.0, split=None):
    """Per-axis cos, sin tables of a 3D rotary embedding: ``((cos_t, sin_t), (cos_h, sin_h), (cos_w, sin_w), (pt, ph, pw))``
    with cos_a, sin_a of shape ``[positions of axis a, pairs of axis a]`` (float32).

    The paper gives neither the split of the head dim over the three axes nor the base frequency, so this
    is only a plausible input for tests and measurements: of the d//2 feature pairs, d//6 go to the height
    and to the width axis each and the rest to time (or ``split = (pt, ph, pw)``); pair i of an axis with n_a
    pairs turns by ``pos * base**(-i / n_a)`` (the rotary formula of Su et al., per axis).
    """
    half = d // 2
    if split is None:
        n_hw = d // 6
        split = (half - 2 * n_hw, n_hw, n_hw)
    assert sum(split) == half
    out = []
    for n_pos, n_a in zip((T, Hh, Ww), split):
        freq = base ** (-np.arange(n_a, dtype=np.float64) / max(n_a, 1))
        theta = np.arange(n_pos, dtype=np.float64)[:, None] * freq[None, :]
        out.append((np.cos(theta).astype(np.float32), np.sin(theta).astype(np.float32)))
    return out[0], out[1], out[2], tuple(split)


def rope_table(T: int, Hh: int, Ww: int, d: int, base: float = 10000.0, split=None):
    """cos, sin tables ``[T*Hh*Ww, d//2]`` (float32) of the same embedding spelled out per token, tokens ordered
    (t, h, w): pairs [0, pt) follow t, [pt, pt+ph) follow h, the rest follow w (see ``rope_axes``)."""
    axes = rope_axes(T, Hh, Ww, d, base, split)
    t, h, w = np.meshgrid(np.arange(T), np.arange(Hh), np.arange(Ww), indexing="ij")
    cos = np.concatenate([axes[a][0][pos.reshape(-1)] for a, pos in enumerate((t, h, w))], axis=1)
    sin = np.concatenate([axes[a][1][pos.reshape(-1)] for a, pos in enumerate((t, h, w))], axis=1)
    assert cos.shape == (T * Hh * Ww, d // 2)
    return np.ascontiguousarray(cos), np.ascontiguousarray(sin)


# ---- inputs of the temporal convolution of the Mix-FFN: x[B, T, HW, D] frames and per-channel taps w[3, D] ----

X_ID, W_ID = 5, 6


@dataclass(frozen=True)
class ConvWorkload:
    name: str
    B: int
    T: int        # frames (all blocks together)
    HW: int       # positions of one frame
    D: int        # channels (the model width)
    seed: int
    T_b: int = 0  # frames per block (0: bidirectional)


# the 480p / 720p latent grids of the attention workloads (21 frames of 30x52 / 45x80 positions), width 2240;
# block-causal: blocks of 3 frames (7 blocks of the 480p clip; a stretch of the 720p stream, batch 2)
CONV_TINY = ConvWorkload("tconv_tiny", B=2, T=5, HW=6, D=16, seed=2001)
CONV_P480 = ConvWorkload("tconv_480p_5s", B=1, T=21, HW=30 * 52, D=2240, seed=2002)
CONV_P720 = ConvWorkload("tconv_720p_5s", B=1, T=21, HW=45 * 80, D=2240, seed=2003)
CONV_AR480 = ConvWorkload("tconv_480p_block_causal", B=1, T=21, HW=30 * 52, D=2240, seed=2004, T_b=3)
CONV_STREAM720 = ConvWorkload("tconv_720p_stream", B=2, T=3 * 8, HW=45 * 80, D=2240, seed=2005, T_b=3)


def conv_frames(w: ConvWorkload, dtype: str = "bf16", t0: int = 0, frames: int | None = None) -> np.ndarray:
    """Frames t0 .. t0+frames of the workload's x, N(0, 1) draws; the same bits whichever range is asked for."""
    frames = w.T - t0 if frames is None else frames
    a = np.empty((w.B, frames, w.HW, w.D), dtype=np.uint16 if dtype == "bf16" else np.float32)
    per = w.HW * w.D
    for b in range(w.B):
        gauss((frames, w.HW, w.D), w.seed, X_ID, start=(b * w.T + t0) * per, dtype=dtype, out=a[b])
    return a


def conv_taps(D: int, seed: int, scale: float = 0.25) -> np.ndarray:
    """Per-channel taps w[3, D] (float32), N(0, scale^2): a trained layer's taps are not known, any values do."""
    return gauss((3, D), seed, W_ID, scale=scale, dtype="f32")
