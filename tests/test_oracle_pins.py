"""Pins for the CPU oracle: what the paper's equations and plain mathematics fix.

The paper prints no worked numerical example of its attention, so the oracle
is pinned to closed forms, a hand-worked example, brute force on tiny inputs,
library routines in special cases, and invariances.  ``test_mutants_are_caught``
then plants mistakes in a copy of the oracle's source (on the CPU) and checks
that these pins reject every one of them.
"""
import os
import subprocess
from fractions import Fraction

import numpy as np
import pytest

import oracle as oracle_mod
import synth

EPS = 1e-6


def _rand(shape, seed, tid=1, dtype="f64"):
    x = synth.gauss(shape, seed, tid, dtype="f32")
    return x.astype(np.float64) if dtype == "f64" else x


def _qkv(B, N, H, d, seed):
    return tuple(_rand((B, N, H, d), seed, t) for t in (1, 2, 3))


# ----------------------------------------------------------------------------- pins
# Each pin takes an Oracle and raises AssertionError when the oracle is wrong.

def pin_hand_worked_example(o):
    """d=2, N=2, worked by hand from Eq. 2 (values in the comments)."""
    q = np.array([[1.0, 1.0], [2.0, 1.0]]).reshape(1, 2, 1, 2)
    k = np.array([[1.0, 2.0], [-3.0, 1.0]]).reshape(1, 2, 1, 2)
    v = np.array([[1.0, 0.0], [0.0, 2.0]]).reshape(1, 2, 1, 2)
    # phi(k1) = (1,2), phi(k2) = (0,1)
    # S = (1,2)^T (1,0) + (0,1)^T (0,2) = [[1,0],[2,2]],  z = (1,3)
    S, z = o.state(k, v)
    assert np.array_equal(S[0, 0], [[1.0, 0.0], [2.0, 2.0]])
    assert np.array_equal(z[0, 0], [1.0, 3.0])
    # q1 = (1,1): num = (3,2), den = 4 ; q2 = (2,1): num = (4,2), den = 5
    for fn in (o.forward, o.quadratic):
        out = fn(q, k, v, 0.0)
        assert np.allclose(out[0, :, 0], [[0.75, 0.5], [0.8, 0.4]], rtol=0, atol=1e-15)
        out = fn(q, k, v, 0.5)
        assert np.allclose(out[0, :, 0], [[3 / 4.5, 2 / 4.5], [4 / 5.5, 2 / 5.5]], rtol=0, atol=1e-15)
    # blocks of one token: token 1 sees only itself: S = [[1,0],[2,0]], z = (1,2): num (3,0), den 3
    for out in (o.quadratic(q, k, v, 0.0, 1), o.block_masked(q, k, v, 0.0, 1)):
        assert np.allclose(out[0, :, 0], [[1.0, 0.0], [0.8, 0.4]], rtol=0, atol=1e-15)
    cache = o.new_cache(1, 1, 2)
    o1 = o.block_step(cache, q[:, :1], k[:, :1], v[:, :1], 0.0)
    o2 = o.block_step(cache, q[:, 1:], k[:, 1:], v[:, 1:], 0.0)
    assert np.allclose(o1[0, 0, 0], [1.0, 0.0], atol=1e-15) and np.allclose(o2[0, 0, 0], [0.8, 0.4], atol=1e-15)
    assert np.array_equal(cache[0][0, 0], [[1.0, 0.0], [2.0, 2.0]]) and np.array_equal(cache[1][0, 0], [1.0, 3.0])


def pin_golden_hand_worked_d2(o):
    """tests/golden/eq2_eq3_hand_worked_d2.txt: Eq. 2 and Eq. 3 worked by hand (derivation in the file)."""
    from parity_util import read_golden

    g = read_golden("eq2_eq3_hand_worked_d2.txt")
    q, k, v = (g[n].reshape(1, 3, 1, 2) for n in ("q", "k", "v"))
    S, z = o.state(k, v)
    assert np.array_equal(S[0, 0], g["S"]) and np.array_equal(z[0, 0], g["z"][0])
    for fn in (o.forward, o.quadratic):
        assert np.allclose(fn(q, k, v, 0.0)[0, :, 0], g["o_bidirectional_eps0"], rtol=0, atol=2e-16)
        assert np.allclose(fn(q, k, v, 0.5)[0, :, 0], g["o_bidirectional_eps_half"], rtol=0, atol=2e-16)
    for out in (o.quadratic(q, k, v, 0.0, 1), o.block_masked(q, k, v, 0.0, 1)):
        assert np.allclose(out[0, :, 0], g["o_blocks_of_one_eps0"], rtol=0, atol=2e-16)
    for out in (o.quadratic(q, k, v, 0.0, 2), o.block_masked(q, k, v, 0.0, 2)):
        assert np.allclose(out[0, :, 0], g["o_blocks_12_3_eps0"], rtol=0, atol=2e-16)
    cache = o.new_cache(1, 1, 2)
    o12 = o.block_step(cache, q[:, :2], k[:, :2], v[:, :2], 0.0)
    o3 = o.block_step(cache, q[:, 2:], k[:, 2:], v[:, 2:], 0.0)
    assert np.allclose(np.concatenate([o12, o3], axis=1)[0, :, 0], g["o_blocks_12_3_eps0"], rtol=0, atol=2e-16)
    assert np.array_equal(cache[0][0, 0], g["S"]) and np.array_equal(cache[1][0, 0], g["z"][0])


def pin_exact_rational(o):
    """Small-integer inputs: the definition evaluated in exact rational arithmetic."""
    N, d = 5, 3
    q = synth.bf16_bits_to_f32(synth.smallint((1, N, 1, d), 7, 1, 3)).astype(np.float64)
    k = synth.bf16_bits_to_f32(synth.smallint((1, N, 1, d), 7, 2, 3)).astype(np.float64)
    v = synth.bf16_bits_to_f32(synth.smallint((1, N, 1, d), 7, 3, 3)).astype(np.float64)
    eps = Fraction(1, 8)
    want = np.zeros((N, d))
    for n in range(N):
        w = [sum(Fraction(max(int(q[0, n, 0, i]), 0) * max(int(k[0, m, 0, i]), 0)) for i in range(d)) for m in range(N)]
        den = sum(w) + eps
        for j in range(d):
            want[n, j] = float(sum(w[m] * int(v[0, m, 0, j]) for m in range(N)) / den)
    for fn in (o.forward, o.quadratic):
        assert np.allclose(fn(q, k, v, float(eps))[0, :, 0], want, rtol=1e-15, atol=1e-15)


def pin_linear_equals_quadratic(o):
    """Re-association only: the linear form reaches the quadratic definition."""
    for (N, d, H, B) in [(1, 1, 1, 1), (2, 2, 2, 1), (3, 1, 1, 2), (17, 32, 2, 2), (192, 32, 4, 1), (40, 7, 3, 1)]:
        q, k, v = _qkv(B, N, H, d, 100 + N + d)
        a, b = o.forward(q, k, v, EPS), o.quadratic(q, k, v, EPS)
        scale = np.abs(b).max() + 1e-300
        assert np.abs(a - b).max() <= 1e-12 * scale, (N, d)


def pin_bf16_decode_and_tiny_config(o):
    """bf16 bit patterns are widened exactly; config 1 (bf16 N(0,1), 4 heads of 32, 192 tokens)."""
    bits = np.array([0x3F80, 0xC000, 0x0000, 0x3E00], dtype=np.uint16).reshape(1, 1, 1, 4)  # 1, -2, 0, 0.125
    ones = np.full((1, 1, 1, 4), 0x3F80, dtype=np.uint16)
    S, z = o.state(ones, bits)  # phi(k)=1 everywhere: every row of S is v
    assert np.array_equal(S[0, 0], np.tile([1.0, -2.0, 0.0, 0.125], (4, 1)))
    w = synth.TINY
    q, k, v = synth.qkv(w)
    a = o.forward(q, k, v, w.eps)
    b = o.quadratic(q, k, v, w.eps)
    assert np.abs(a - b).max() <= 1e-12 * np.abs(b).max()
    f = lambda x: synth.bf16_bits_to_f32(x).astype(np.float64)
    c = o.forward(f(q), f(k), f(v), w.eps)
    assert np.array_equal(a, c)


def pin_constant_v(o):
    """v_n = c for all n  =>  o_n = c * D/(D+eps), D = phi(q_n).z."""
    B, N, H, d = 1, 33, 2, 8
    q, k, _ = _qkv(B, N, H, d, 5)
    c = _rand((d,), 6)
    v = np.broadcast_to(c, (B, N, H, d)).copy()
    out = o.forward(q, k, v, EPS)
    _, z = o.state(k, v)
    D = np.einsum("bnhi,bhi->bnh", np.maximum(q, 0), z)
    want = c[None, None, None, :] * (D / (D + EPS))[..., None]
    assert np.allclose(out, want, rtol=1e-12, atol=1e-15)
    # z itself: column sums of relu(k)
    assert np.allclose(z, np.maximum(k, 0).sum(axis=1), rtol=1e-13)


def pin_single_token(o):
    """N = 1: o = v * D/(D+eps) with D = phi(q).phi(k); D = 0 gives exactly 0."""
    d = 6
    q = np.array([1.0, -2.0, 0.5, 0.0, 3.0, -1.0]).reshape(1, 1, 1, d)
    k = np.array([2.0, 5.0, -1.0, 4.0, 0.25, -7.0]).reshape(1, 1, 1, d)
    v = _rand((1, 1, 1, d), 9)
    D = 1.0 * 2.0 + 3.0 * 0.25
    for eps in (EPS, 0.3):
        assert np.allclose(o.forward(q, k, v, eps), v * D / (D + eps), rtol=1e-14)
    out = o.forward(-np.abs(q), k, v, EPS)
    assert np.array_equal(out, np.zeros_like(out)) and not np.isnan(out).any()
    out = o.forward(q, -np.abs(k), v, EPS)  # empty state
    assert np.array_equal(out, np.zeros_like(out))


def pin_one_hot_is_segment_mean(o):
    """One-hot q and k turn the op into a per-class mean of V (numpy bincount)."""
    N, d, C = 200, 5, 4
    a = synth.index((N,), 11, 1, C)  # class of each query
    c = synth.index((N,), 11, 2, C)  # class of each key
    feat = C + 2  # two never-used feature slots
    q = np.zeros((1, N, 1, feat)); q[0, np.arange(N), 0, a] = 1.0
    k = np.zeros((1, N, 1, feat)); k[0, np.arange(N), 0, c] = 3.0  # key magnitude cancels
    v = np.zeros((1, N, 1, feat)); v[0, :, 0, :d] = synth.bf16_bits_to_f32(synth.smallint((N, d), 11, 3, 5))
    out = o.forward(q, k, v, 0.0)
    cnt = np.bincount(c, minlength=C)
    for j in range(d):
        mean = np.bincount(c, weights=v[0, :, 0, j], minlength=C) / cnt
        assert np.allclose(out[0, :, 0, j], mean[a], rtol=1e-14, atol=1e-15)


def pin_invariances(o):
    B, N, H, d = 2, 29, 3, 10
    q, k, v = _qkv(B, N, H, d, 21)
    v2 = _rand((B, N, H, d), 22, 3)
    base = o.forward(q, k, v, 0.0)
    # linear in V
    assert np.allclose(o.forward(q, k, v + v2, 0.0), base + o.forward(q, k, v2, 0.0), rtol=1e-11, atol=1e-13)
    # positive scaling of q or k cancels (eps = 0)
    assert np.allclose(o.forward(2.0 * q, k, v, 0.0), base, rtol=1e-12, atol=1e-14)
    assert np.allclose(o.forward(q, 0.25 * k, v, 0.0), base, rtol=1e-12, atol=1e-14)
    # with eps the scaling shows exactly as eps/scale
    assert np.allclose(o.forward(4.0 * q, k, v, 4.0 * 0.1), o.forward(q, k, v, 0.1), rtol=1e-12, atol=1e-14)
    # joint permutation of (k, v) rows changes nothing; permuting q rows permutes o rows
    p = np.argsort(synth.index((N,), 23, 1, 1 << 20))
    assert np.allclose(o.forward(q, np.ascontiguousarray(k[:, p]), np.ascontiguousarray(v[:, p]), EPS), o.forward(q, k, v, EPS), rtol=1e-11, atol=1e-13)
    assert np.array_equal(o.forward(np.ascontiguousarray(q[:, p]), k, v, EPS), o.forward(q, k, v, EPS)[:, p])
    # heads and batches are independent
    one = o.forward(q[1:, :, 2:3], k[1:, :, 2:3], v[1:, :, 2:3], EPS)
    assert np.array_equal(one, o.forward(q, k, v, EPS)[1:, :, 2:3])


def pin_sign(o):
    """Only the positive parts of q and k matter."""
    B, N, H, d = 1, 23, 2, 9
    q, k, v = _qkv(B, N, H, d, 31)
    base = o.forward(q, k, v, EPS)
    assert np.array_equal(o.forward(np.maximum(q, 0), k, v, EPS), base)
    assert np.array_equal(o.forward(q, np.maximum(k, 0), v, EPS), base)
    assert np.array_equal(o.forward(np.where(q < 0, 7.0 * q, q), np.where(k < 0, 3.0 * k, k), v, EPS), base)
    q2 = q.copy(); q2[0, 5] = -np.abs(q2[0, 5])
    out = o.forward(q2, k, v, EPS)
    assert np.array_equal(out[0, 5], np.zeros((H, d)))
    # negative v passes through with its sign
    assert np.allclose(o.forward(q, k, -v, EPS), -base, rtol=1e-14)


def pin_convexity(o):
    """Weights are >= 0 and sum to 1 (eps -> 0): outputs lie within the range of V."""
    B, N, H, d = 1, 50, 2, 6
    q, k, v = _qkv(B, N, H, d, 41)
    out = o.forward(q, k, v, 0.0)
    lo, hi = v.min(axis=1, keepdims=True), v.max(axis=1, keepdims=True)
    ok = np.isfinite(out)
    assert ((out >= lo - 1e-12) & (out <= hi + 1e-12))[ok].all() and ok.mean() > 0.9


def pin_block_forms_agree(o):
    """Stepping a cache == one-shot prefix form == masked quadratic definition."""
    for (B, H, d, T_b, M, tail) in [(1, 2, 4, 5, 3, 0), (2, 1, 3, 1, 4, 0), (1, 3, 8, 6, 3, 2)]:
        N = T_b * M + tail
        q, k, v = _qkv(B, N, H, d, 50 + T_b)
        brute = o.quadratic(q, k, v, EPS, T_b)
        pre = o.block_masked(q, k, v, EPS, T_b)
        cache = o.new_cache(B, H, d)
        outs = []
        for n0 in range(0, N, T_b):
            sl = slice(n0, min(n0 + T_b, N))
            outs.append(o.block_step(cache, np.ascontiguousarray(q[:, sl]), np.ascontiguousarray(k[:, sl]),
                                     np.ascontiguousarray(v[:, sl]), EPS))
            assert cache[0].nbytes + cache[1].nbytes == o.cache_bytes(B, H, d)
        stepped = np.concatenate(outs, axis=1)
        sc = np.abs(brute).max()
        assert np.abs(pre - brute).max() <= 1e-12 * sc
        assert np.abs(stepped - brute).max() <= 1e-12 * sc
        # block identities: first block == forward on it alone; last block == tail of the bidirectional forward;
        # final cache == state of the whole sequence; one block == forward
        assert np.allclose(stepped[:, :T_b], o.forward(q[:, :T_b].copy(), k[:, :T_b].copy(), v[:, :T_b].copy(), EPS),
                           rtol=1e-12, atol=1e-14)
        last0 = (N - 1) // T_b * T_b
        assert np.allclose(stepped[:, last0:], o.forward(q, k, v, EPS)[:, last0:], rtol=1e-11, atol=1e-13)
        S, z = o.state(k, v)
        assert np.allclose(cache[0], S, rtol=1e-12, atol=1e-13) and np.allclose(cache[1], z, rtol=1e-12, atol=1e-13)
        assert np.allclose(o.block_masked(q, k, v, EPS, N), o.forward(q, k, v, EPS), rtol=1e-13, atol=1e-15)
        # a later block must not leak into an earlier one
        k2, v2 = k.copy(), v.copy()
        k2[:, T_b:] = np.abs(k2[:, T_b:]) + 1.0; v2[:, T_b:] += 5.0
        assert np.array_equal(o.block_masked(q, k2, v2, EPS, T_b)[:, :T_b], pre[:, :T_b])
        assert not np.allclose(o.block_masked(q, k2, v2, EPS, T_b)[:, T_b:], pre[:, T_b:])


def pin_cache_size_constant(o):
    """Table 1: cache memory is O(D^2), independent of the number of blocks."""
    B, H, d = 1, 2, 16
    cache = o.new_cache(B, H, d)
    sizes = []
    for blk in range(80):
        q, k, v = _qkv(B, 3, H, d, 60 + blk)
        o.block_step(cache, q, k, v, EPS, want_o=False)
        if blk + 1 in (1, 7, 80):
            sizes.append(cache[0].nbytes + cache[1].nbytes)
    assert sizes == [B * H * (d * d + d) * 8] * 3 == [o.cache_bytes(B, H, d)] * 3
    assert o.cache_bytes(2, 20, 112) == 2 * 20 * (112 * 112 + 112) * 8


def pin_strides_and_rows(o):
    """[B,H,N,d] storage viewed as [B,N,H,d]; apply_rows == rows of forward."""
    B, N, H, d = 2, 11, 3, 4
    q, k, v = _qkv(B, N, H, d, 71)
    base = o.forward(q, k, v, EPS)
    tr = lambda x: np.ascontiguousarray(x.transpose(0, 2, 1, 3)).transpose(0, 2, 1, 3)
    assert np.array_equal(o.forward(tr(q), tr(k), tr(v), EPS), base)
    S, z = o.state(k, v)
    rows = np.array([10, 0, 3])
    assert np.array_equal(o.apply_rows(q, S, z, EPS, rows), base[:, rows])
    # state transposition check: S[i][j] pairs key feature i with value feature j
    k1 = np.zeros((1, 1, 1, 3)); k1[..., 0] = 2.0
    v1 = np.zeros((1, 1, 1, 3)); v1[..., 2] = 5.0
    S1, z1 = o.state(k1, v1)
    want = np.zeros((3, 3)); want[0, 2] = 10.0
    assert np.array_equal(S1[0, 0], want) and np.array_equal(z1[0, 0], [2.0, 0.0, 0.0])


def _angles(N, half, seed, scale=3.0):
    th = synth.gauss((N, half), seed, 7, dtype="f32").astype(np.float64) * scale
    return np.cos(th), np.sin(th), th


def pin_rope_closed_form_d2(o):
    """d = 2, phi(q) = phi(k) = (1, 0): the rotated dot product is cos(theta_n - theta_m), the plain one is 1,
    so o_n = sum_m cos(theta_n - theta_m) v_m / (N + eps)  (Eq. 2, right-hand form)."""
    N = 5
    th = np.array([0.0, 0.3, -1.1, 2.0, np.pi / 2])
    q = np.zeros((1, N, 1, 2)); q[..., 0] = 1.0; q[..., 1] = -2.0      # the negative entry is cut by the ReLU
    k = q.copy()
    v = _rand((1, N, 1, 2), 81, 3)
    want = (np.cos(th[:, None] - th[None, :]) @ v[0, :, 0]) / (N + 0.25)
    for quad in (False, True):
        out = o.rope_forward(q, k, v, np.cos(th)[:, None], np.sin(th)[:, None], 0.25, quadratic=quad)
        assert np.allclose(out[0, :, 0], want, rtol=0, atol=1e-14)
    # table column p belongs to feature pair (2p, 2p+1): with d = 4 and only features 0, 1 alive, angles in
    # column 0 act as above and angles in column 1 do nothing
    q4 = np.zeros((1, N, 1, 4)); q4[..., 0] = 1.0
    v4 = _rand((1, N, 1, 4), 82, 3)
    zero = np.zeros(N)
    out = o.rope_forward(q4, q4.copy(), v4, np.stack([np.cos(th), np.cos(zero)], 1), np.stack([np.sin(th), np.sin(zero)], 1), 0.25)
    assert np.allclose(out[0, :, 0], (np.cos(th[:, None] - th[None, :]) @ v4[0, :, 0]) / (N + 0.25), rtol=0, atol=1e-14)
    out = o.rope_forward(q4, q4.copy(), v4, np.stack([np.cos(zero), np.cos(th)], 1), np.stack([np.sin(zero), np.sin(th)], 1), 0.25)
    assert np.allclose(out[0, :, 0], np.broadcast_to(v4[0, :, 0].sum(0) / (N + 0.25), (N, 4)), rtol=0, atol=1e-14)
    # a quarter turn on the key only: (1,0) -> (0,1), orthogonal to the unrotated query: numerator 0, denominator not
    th2 = np.array([0.0, np.pi / 2])
    out = o.rope_forward(q[:, :2].copy(), k[:, :2].copy(), np.ones((1, 2, 1, 2)), np.cos(th2)[:, None], np.sin(th2)[:, None], 0.0)
    assert np.allclose(out[0, 0, 0], [0.5, 0.5], atol=1e-14) and np.allclose(out[0, 1, 0], [0.5, 0.5], atol=1e-14)
    # rotation direction: (a, b) -> (a c - b s, a s + b c).  k = (0, 1) turned by +90 deg becomes (-1, 0)
    qd = np.array([1.0, 0.0]).reshape(1, 1, 1, 2); kd = np.array([0.0, 1.0]).reshape(1, 1, 1, 2)
    q2 = np.concatenate([qd, qd], 1); k2 = np.concatenate([kd, kd], 1); v2 = np.array([[1.0, 0.0], [0.0, 1.0]]).reshape(1, 2, 1, 2)
    out = o.rope_forward(q2, k2, v2, np.array([[1.0], [0.0]]), np.array([[0.0], [1.0]]), 1.0)
    # token 0 (angle 0): rotated q = (1,0); rotated keys: (0,1) and (-1,0): weights 0 and -1; plain weights 0, 0
    assert np.allclose(out[0, 0, 0], [0.0, -1.0], atol=1e-14)


def pin_rope_block_causal_closed_form_d2(o):
    """d = 2, phi(q) = phi(k) = (1, 0), blocks of T_b tokens: token n sees the tokens of its own and of earlier
    blocks, the rotated dot product is cos(theta_n - theta_m) and the plain one is 1, so
    o_n = sum_{m visible} cos(theta_n - theta_m) v_m / (count_n + eps)  (Eq. 3's running sums on Eq. 2's
    right-hand form).  Fixes the block-causal rotary form against the mathematics in all three ways the oracle
    computes it: block by block, masked brute force, and cached steps on a caller-held cache."""
    N, T_b, eps = 11, 4, 0.5                      # blocks of 4, 4 and 3 tokens
    th = np.array([0.0, 0.3, -1.1, 2.0, np.pi / 2, -0.4, 1.7, 0.9, -2.5, 0.05, 3.0])
    q = np.zeros((1, N, 1, 2)); q[..., 0] = 1.0; q[..., 1] = -3.0     # the negative entry is cut by the ReLU
    k = q.copy()
    v = _rand((1, N, 1, 2), 91, 3)
    blk = np.arange(N) // T_b
    visible = blk[None, :] <= blk[:, None]                            # [n, m]
    want = ((np.cos(th[:, None] - th[None, :]) * visible) @ v[0, :, 0]) / (visible.sum(1) + eps)[:, None]
    cs, sn = np.cos(th)[:, None], np.sin(th)[:, None]
    assert np.allclose(o.rope_forward(q, k, v, cs, sn, eps, T_b=T_b)[0, :, 0], want, rtol=0, atol=1e-14)
    assert np.allclose(o.rope_forward(q, k, v, cs, sn, eps, quadratic=True, T_b=T_b)[0, :, 0], want, rtol=0, atol=1e-14)
    cache = o.new_cache(1, 1, 2)
    for n0 in range(0, N, T_b):
        sl = slice(n0, min(n0 + T_b, N))
        args = (q[:, sl].copy(), k[:, sl].copy(), v[:, sl].copy(), cs[sl], sn[sl], eps)
        # a denoising step of Algorithm 1 reads the cache without committing: the step on a copy
        peek = o.rope_block_step((cache[0].copy(), cache[1].copy()), *args)
        before = (cache[0].copy(), cache[1].copy())
        out = o.rope_block_step(cache, *args)
        assert np.array_equal(peek, out)
        assert np.allclose(out[0, :, 0], want[sl], rtol=0, atol=1e-14)
        assert not np.array_equal(before[1], cache[1])                # the committing step did change the cache
    # the cache after the last block, in closed form: z = (N, 0); S = sum_m (cos, sin)(theta_m)^T v_m
    S, z = cache
    assert np.array_equal(z[0, 0], [N, 0.0])
    assert np.allclose(S[0, 0], np.stack([np.cos(th), np.sin(th)], 0) @ v[0, :, 0], rtol=0, atol=1e-14)
    # commit only (no output) leaves the same cache
    c2 = o.new_cache(1, 1, 2)
    for n0 in range(0, N, T_b):
        sl = slice(n0, min(n0 + T_b, N))
        assert o.rope_block_step(c2, q[:, sl].copy(), k[:, sl].copy(), v[:, sl].copy(), cs[sl], sn[sl], eps, want_o=False) is None
    assert np.array_equal(c2[0], S) and np.array_equal(c2[1], z)


def pin_rope_steps_equal_one_shot(o):
    """Cached rotary steps over several heads and batch entries equal the one-shot block-causal form, and a
    step's table rows are the block's own: shifting them by one token changes the result."""
    B, N, H, d, T_b = 2, 10, 3, 6, 4
    q, k, v = _qkv(B, N, H, d, 95)
    cs, sn, _ = _angles(N, d // 2, 96)
    ref = o.rope_forward(q, k, v, cs, sn, EPS, T_b=T_b)
    cache = o.new_cache(B, H, d)
    for n0 in range(0, N, T_b):
        sl = slice(n0, min(n0 + T_b, N))
        out = o.rope_block_step(cache, q[:, sl].copy(), k[:, sl].copy(), v[:, sl].copy(), cs[sl], sn[sl], EPS)
        assert np.allclose(out, ref[:, sl], rtol=1e-12, atol=1e-13)
    sl = slice(4, 8)
    c0 = o.new_cache(B, H, d)
    a = o.rope_block_step(c0, q[:, sl].copy(), k[:, sl].copy(), v[:, sl].copy(), cs[sl], sn[sl], EPS)
    c1 = o.new_cache(B, H, d)
    b = o.rope_block_step(c1, q[:, sl].copy(), k[:, sl].copy(), v[:, sl].copy(), cs[5:9], sn[5:9], EPS)
    assert np.abs(a - b).max() > 1e-3
    # units are independent and land in their own slice of the cache
    c3 = o.new_cache(1, 1, d)
    o.rope_block_step(c3, q[1:, sl, 2:].copy(), k[1:, sl, 2:].copy(), v[1:, sl, 2:].copy(), cs[sl], sn[sl], EPS)
    assert np.array_equal(c3[0][0, 0], c0[0][1, 2]) and np.array_equal(c3[1][0, 0], c0[1][1, 2])


def pin_rope_reduces_to_plain(o):
    """Zero angles, or one common angle per feature pair for all tokens (relative angle zero), give Eq. 2
    without rotary factors: the numerator only sees angle differences and the denominator sees none."""
    B, N, H, d = 2, 9, 2, 6
    q, k, v = _qkv(B, N, H, d, 83)
    plain = o.forward(q, k, v, EPS)
    one, zero = np.ones((N, d // 2)), np.zeros((N, d // 2))
    assert np.array_equal(o.rope_forward(q, k, v, one, zero, EPS), plain)
    delta = np.array([0.7, -2.0, 1.3])
    cs, sn = np.broadcast_to(np.cos(delta), (N, 3)), np.broadcast_to(np.sin(delta), (N, 3))
    assert np.allclose(o.rope_forward(q, k, v, cs, sn, EPS), plain, rtol=1e-12, atol=1e-13)
    # ... and with real angles the result differs from the plain one
    cs, sn, _ = _angles(N, 3, 84)
    assert np.abs(o.rope_forward(q, k, v, cs, sn, EPS) - plain).max() > 1e-3


def pin_rope_linear_equals_quadratic_and_shift(o):
    for (B, N, H, d, seed) in [(1, 1, 1, 2, 85), (2, 7, 3, 4, 86), (1, 33, 2, 14, 87), (1, 12, 1, 5, 88)]:
        q, k, v = _qkv(B, N, H, d, seed)
        cs, sn, th = _angles(N, d // 2, seed + 100)
        lin = o.rope_forward(q, k, v, cs, sn, EPS)
        quad = o.rope_forward(q, k, v, cs, sn, EPS, quadratic=True)
        assert np.allclose(lin, quad, rtol=1e-11, atol=1e-12)
        # only angle differences matter: a common offset per pair changes nothing
        off = np.linspace(-1.0, 2.0, d // 2)
        assert np.allclose(o.rope_forward(q, k, v, np.cos(th + off), np.sin(th + off), EPS), lin, rtol=1e-11, atol=1e-12)
        # the denominator is the plain one: scaling V scales the output, and sum_m w_den is that of the plain form
        ones = np.ones_like(v)
        den_ratio = o.rope_forward(q, k, ones, cs, sn, EPS)          # = sum_m w_num / (sum_m w_den + eps), same in every column
        assert np.allclose(den_ratio, den_ratio[..., :1], rtol=1e-12, atol=1e-13)
    # block-causal: cached block-by-block == masked brute force; one block == bidirectional; last block sees all
    q, k, v = _qkv(2, 14, 2, 6, 91)
    cs, sn, _ = _angles(14, 3, 92)
    for T_b in (2, 4, 5, 14, 20):
        assert np.allclose(o.rope_forward(q, k, v, cs, sn, 1e-3, T_b=T_b),
                           o.rope_forward(q, k, v, cs, sn, 1e-3, quadratic=True, T_b=T_b), rtol=1e-9, atol=1e-10)
    full = o.rope_forward(q, k, v, cs, sn, EPS)
    assert np.allclose(o.rope_forward(q, k, v, cs, sn, EPS, T_b=14), full, rtol=1e-12, atol=1e-13)
    assert np.allclose(o.rope_forward(q, k, v, cs, sn, EPS, T_b=5)[:, 10:], full[:, 10:], rtol=1e-11, atol=1e-12)
    # ... and a block is blind to later blocks
    k2, v2 = k.copy(), v.copy(); k2[:, 8:] += 1.0; v2[:, 8:] -= 2.0
    assert np.array_equal(o.rope_forward(q, k, v, cs, sn, EPS, T_b=4)[:, :8], o.rope_forward(q, k2, v2, cs, sn, EPS, T_b=4)[:, :8])
    # each head and batch entry is independent, the table is shared
    q, k, v = _qkv(2, 6, 2, 4, 89)
    cs, sn, _ = _angles(6, 2, 90)
    full = o.rope_forward(q, k, v, cs, sn, EPS)
    part = o.rope_forward(q[1:, :, 1:].copy(), k[1:, :, 1:].copy(), v[1:, :, 1:].copy(), cs, sn, EPS)
    assert np.array_equal(full[1:, :, 1:], part)


PINS = [pin_hand_worked_example, pin_golden_hand_worked_d2, pin_exact_rational, pin_linear_equals_quadratic, pin_bf16_decode_and_tiny_config,
        pin_constant_v, pin_single_token, pin_one_hot_is_segment_mean, pin_invariances, pin_sign, pin_convexity,
        pin_block_forms_agree, pin_cache_size_constant, pin_strides_and_rows, pin_rope_closed_form_d2,
        pin_rope_reduces_to_plain, pin_rope_linear_equals_quadratic_and_shift, pin_rope_block_causal_closed_form_d2,
        pin_rope_steps_equal_one_shot]


@pytest.mark.parametrize("pin", PINS, ids=lambda f: f.__name__)
def test_pin(orc, pin):
    pin(orc)


# ----------------------------------------------------------------------------- mutation test
# (old text, new text): each plants one plausible mistake in a copy of the oracle source.
MUTANTS = {
    "relu_dropped": ("return x > 0.0 ? x : 0.0;", "return x;"),
    "relu_is_abs": ("return x > 0.0 ? x : 0.0;", "return x > 0.0 ? x : -x;"),
    "z_scaled": ("z[i] += kp;", "z[i] += 0.5 * kp;"),
    "state_transposed": ("Srow[j] += kp * load_elem(v, s->dtype, base + j);",
                         "S[j * d + i] += kp * load_elem(v, s->dtype, base + j);"),
    "apply_transposed": ("for (int64_t j = 0; j < d; ++j) o_row[j] += qp * Srow[j];",
                         "for (int64_t j = 0; j < d; ++j) o_row[j] += qp * S[j * d + i];"),
    "eps_dropped": ("  den += eps;\n", "\n"),
    "eps_inside_sum": ("    den += qp * z[i];", "    den += qp * z[i] + eps;"),
    "den_without_q": ("den += qp * z[i];", "den += z[i];"),
    "q_relu_dropped": ("const double qp = relu(load_elem(q, s->dtype, base + i));",
                       "const double qp = load_elem(q, s->dtype, base + i);"),
    "k_relu_dropped_linear": ("const double kp = relu(load_elem(k, s->dtype, base + i));",
                              "const double kp = load_elem(k, s->dtype, base + i);"),
    "k_relu_dropped_quadratic": ("* relu(load_elem(k, s->dtype, kb + i));", "* load_elem(k, s->dtype, kb + i);"),
    "mask_excludes_own_block": ("(m / T_b) > (n / T_b)", "(m / T_b) >= (n / T_b)"),
    "mask_token_causal": ("(m / T_b) > (n / T_b)", "m > n"),
    "step_applies_before_commit": (
        "    accumulate_state(s, k, v, b, h, 0, s->N, S + u * d * d, z + u * d);\n    if (o)\n"
        "      for (int64_t n = 0; n < s->N; ++n)\n"
        "        apply_token(s, q, b, n, h, S + u * d * d, z + u * d, eps, o + ((b * s->N + n) * s->H + h) * d);\n",
        "    if (o)\n      for (int64_t n = 0; n < s->N; ++n)\n"
        "        apply_token(s, q, b, n, h, S + u * d * d, z + u * d, eps, o + ((b * s->N + n) * s->H + h) * d);\n"
        "    accumulate_state(s, k, v, b, h, 0, s->N, S + u * d * d, z + u * d);\n"),
    "prefix_not_accumulated": ("      accumulate_state(s, k, v, b, h, n0, n1, S, z);",
                               "      memset(S, 0, sizeof(double) * (d * d + d));\n"
                               "      accumulate_state(s, k, v, b, h, n0, n1, S, z);"),
    "bf16_shift": ("[idx] << 16;", "[idx] << 15;"),
    "strides_swapped": ("n * s->stride_n + h * s->stride_h", "h * s->stride_n + n * s->stride_h"),
    "v_index_uses_i": ("Srow[j] += kp * load_elem(v, s->dtype, base + j);", "Srow[j] += kp * load_elem(v, s->dtype, base + i);"),
    "cache_bytes_grow": ("return B * H * (d * d + d) * (int64_t)sizeof(double);", "return B * H * (d * d) * (int64_t)sizeof(double);"),
    "state_not_zeroed": ("    memset(Su, 0, sizeof(double) * d * d);\n", ""),
    "rope_before_relu_sign": ("rot[2 * p] = plain[2 * p] * c - plain[2 * p + 1] * t;", "rot[2 * p] = plain[2 * p] * c + plain[2 * p + 1] * t;"),
    "rope_pairs_half_split": ("const double c = cs[n * half + p], t = sn[n * half + p];", "const double c = cs[n * half + (p + 1) % half], t = sn[n * half + (p + 1) % half];"),
    "rope_in_denominator_linear": ("        z[i] += plain[i];\n", "        z[i] += rot[i];\n"),
    "rope_den_uses_rotated_query": ("        den += plain[i] * z[i];\n", "        den += rot[i] * z[i];\n"),
    "rope_state_from_plain_keys": ("S[i * d + j] += rot[i] * load_elem(v, s->dtype, base + j);", "S[i * d + j] += plain[i] * load_elem(v, s->dtype, base + j);"),
    "rope_quadratic_den_rotated": ("wden += qp[i] * kp[i];", "wden += qr[i] * kr[i];"),
    "rope_block_mask_off": ("if (T_b > 0 && (m / T_b) > (n / T_b)) continue; /* later block: not visible (T_b <= 0: no mask) */",
                            "if (T_b > 0 && (m / T_b) >= (n / T_b)) continue;"),
    "rope_block_reads_before_commit": ("  for (int64_t n = n0; n < n1; ++n) { /* commit the block ... */",
                                       "  for (int64_t n = n0; n < n0; ++n) { /* commit the block ... */"),
    "rope_block_forgets_past": ("      rope_block(s, q, k, v, cs, sn, b, h, n0, n1, eps, S, z, z + d, z + 2 * d, o);",
                                "      memset(S, 0, sizeof(double) * (d * d + d));\n"
                                "      rope_block(s, q, k, v, cs, sn, b, h, n0, n1, eps, S, z, z + d, z + 2 * d, o);"),
    "rope_step_unit_offset": ("S + u * d * d, z + u * d, tmp, tmp + d, o);", "S + u * d, z + u * d, tmp, tmp + d, o);"),
    "rope_step_cache_zeroed": ("    double* tmp = (double*)calloc((size_t)(2 * d), sizeof(double));\n    rope_block(",
                               "    double* tmp = (double*)calloc((size_t)(2 * d), sizeof(double));\n"
                               "    memset(z + u * d, 0, sizeof(double) * d);\n    rope_block("),
    "rope_step_first_head_only": ("u / s->H, u % s->H, 0, s->N, eps,", "u / s->H, 0, 0, s->N, eps,"),
    "rope_token_index": ("rope_features(s, k, base, cs, sn, n, plain, rot);", "rope_features(s, k, base, cs, sn, 0, plain, rot);"),
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_mutants_are_caught(tmp_path, name):
    old, new = MUTANTS[name]
    src = open(oracle_mod.SOURCE).read()
    assert src.count(old) >= 1, f"mutation site for {name} not found in the oracle source"
    p = tmp_path / f"mutant_{name}.c"
    p.write_text(src.replace(old, new))
    so = str(tmp_path / f"mutant_{name}.so")
    subprocess.check_call(["gcc", *oracle_mod.CFLAGS, "-o", so, str(p), "-lm"])
    mutant = oracle_mod.Oracle(so)
    caught = []
    for pin in PINS:
        try:
            with np.errstate(all="ignore"):
                pin(mutant)
        except AssertionError:
            caught.append(pin.__name__)
    assert caught, f"no pin rejects the planted mistake '{name}'"
