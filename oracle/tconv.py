"""fp64 CPU oracle of the temporal convolution of the Mix-FFN and of its block-causal form.

TEST INFRASTRUCTURE ONLY.  Nothing under the product package may import this module.

What the paper fixes (Sec. 3.1 "Mix-FFN with Spatial-Temporal Mixture", Sec. 3.2 "Block Causal
Mix-FFN", Algorithm 1's conv cache f): a 1D convolution over the frame axis with kernel size 3 is added
to the end of the Mix-FFN through a shortcut connection; in the block-causal model an all-zero frame is
appended to every block (nothing of a later block is seen) and the last frame of the previous block,
kept in a cache of one frame, is put in front of the block.

What it leaves open, and the reading taken here: the taps act per channel (w[tau][c], tau = 0 the
previous frame, 1 the frame itself, 2 the next one: a cross-correlation, the deep-learning
convention), there is no bias, the frames before the first one are zero, and the shortcut adds the
unconvolved input: y_t = x_t + w0 * x_{t-1} + w1 * x_t + w2 * x_{t+1}.

Tensors are numpy arrays x[B, T, HW, D] (frames, positions of a frame, channels), widened to fp64
exactly; taps w[3, D].  Loops run over frames; each frame is one numpy expression.
"""
from __future__ import annotations

import numpy as np


def widen(a: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) / float32 / float64 -> float64, exactly."""
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def frame_out(prev, cur, nxt, w):
    """One output frame: the shortcut plus the three taps (Sec. 3.1)."""
    return cur + w[0] * prev + w[1] * cur + w[2] * nxt


def tconv_bidirectional(x, w):
    """The short-video model's layer: every frame sees its two neighbours, zeros beyond both ends."""
    x, w = widen(x), np.asarray(w, dtype=np.float64)
    B, T, HW, D = x.shape
    zero = np.zeros((B, HW, D))
    y = np.empty_like(x)
    for t in range(T):
        prev = x[:, t - 1] if t > 0 else zero
        nxt = x[:, t + 1] if t + 1 < T else zero
        y[:, t] = frame_out(prev, x[:, t], nxt, w)
    return y


def tconv_block_masked(x, w, T_b):
    """Block-causal form in one shot (Sec. 3.2): frames are grouped into blocks of T_b frames; the frame
    after a block's last one is the all-zero padding frame, the frame before a block's first one is the
    last frame of the block before it (zeros before the first block)."""
    x, w = widen(x), np.asarray(w, dtype=np.float64)
    B, T, HW, D = x.shape
    zero = np.zeros((B, HW, D))
    y = np.empty_like(x)
    for t in range(T):
        prev = x[:, t - 1] if t > 0 else zero                    # same block, or the block before: both visible
        last_of_block = (t + 1) % T_b == 0 or t + 1 == T
        nxt = zero if last_of_block else x[:, t + 1]
        y[:, t] = frame_out(prev, x[:, t], nxt, w)
    return y


def new_cache(B, HW, D):
    """The conv cache f of Algorithm 1 before the first block: one all-zero frame."""
    return np.zeros((B, HW, D))


def tconv_block_step(x_blk, w, cache, commit=True):
    """One block with the cached frame in front and the zero frame behind (Sec. 3.2, Algorithm 1).
    Returns (y_blk, cache'): with commit the cache becomes the block's last frame (the clean block of
    Algorithm 1), without it the cache is returned as it was (a denoising step only reads it)."""
    x, w = widen(x_blk), np.asarray(w, dtype=np.float64)
    B, T, HW, D = x.shape
    padded = np.concatenate([cache[:, None], x, np.zeros((B, 1, HW, D))], axis=1)   # [f, x_0 .. x_{T-1}, 0]
    y = np.empty_like(x)
    for t in range(T):
        y[:, t] = frame_out(padded[:, t], padded[:, t + 1], padded[:, t + 2], w)
    new = x[:, T - 1].copy() if (commit and T > 0) else cache
    return y, new


def cache_elems(B, HW, D):
    """Elements the conv cache holds, whatever the number of blocks seen: one frame."""
    return B * HW * D
