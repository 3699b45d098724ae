"""Tolerance checks and tensor plumbing shared by the GPU parity tests."""
import numpy as np


def to_dev(bits_or_f32, device="cuda"):
    """numpy uint16 (bf16 bits) or float32 -> torch tensor on the device."""
    import torch

    a = np.ascontiguousarray(bits_or_f32)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    assert a.dtype == np.float32
    return torch.from_numpy(a).to(device)


def to_f64(t):
    """torch tensor (bf16 / f32) -> numpy float64, exactly."""
    import torch

    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def assert_parity_bf16(got, ref, what="", rms_rel=1e-2):
    """bf16 I/O with fp32 accumulation.  `got`, `ref`: float64 [B, n, H, d].
    rms_rel: weight of the head's RMS in bar 2 (1e-2; the rotary tensor-core path, which also rounds the rotated
    queries and keys to bf16, is given 1.5e-2 where hundreds of thousands of elements are compared: its per-element
    error has a standard deviation of about 0.2 % of the RMS, and the largest of 6e5 samples reaches five of them).

    1. the stated bar: |delta| <= 1e-2 + 1e-2*|ref| per element;
    2. the same with the absolute term scaled by the head's RMS of ref, because with zero-mean V the
       outputs are far smaller than 1e-2 and bar 1 alone would accept all-zeros;
    3. relative L2 error per (batch, head) <= 5e-3.
    """
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    delta = np.abs(got - ref)
    assert (delta <= 1e-2 + 1e-2 * np.abs(ref)).all(), f"{what}: stated tolerance, max delta {delta.max():.3e}"
    rms = np.sqrt((ref ** 2).mean(axis=(1, 3), keepdims=True))
    bad = delta > rms_rel * rms + 1e-2 * np.abs(ref)
    assert not bad.any(), (f"{what}: RMS-scaled tolerance: {bad.sum()} of {bad.size} elements, "
                           f"worst ratio {(delta / (rms_rel * rms + 1e-2 * np.abs(ref) + 1e-300)).max():.3f}")
    num = np.sqrt((delta ** 2).sum(axis=(1, 3)))
    den = np.sqrt((ref ** 2).sum(axis=(1, 3)))
    ok = num <= 5e-3 * den + 1e-300
    assert ok.all(), f"{what}: relative L2 per head up to {(num / (den + 1e-300)).max():.3e}"


def assert_parity_f32(got, ref, what="", rel=1e-5):
    """fp32 I/O path: |delta| <= 1e-5 * (|ref| + rms_head(ref))."""
    assert got.shape == ref.shape
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    rms = np.sqrt((ref ** 2).mean(axis=(1, 3), keepdims=True))
    delta = np.abs(got - ref)
    bound = rel * (np.abs(ref) + rms)
    assert (delta <= bound).all(), f"{what}: worst ratio {(delta / (bound + 1e-300)).max():.3f}"


def assert_state_close(state_gpu, S, z, rel=1e-5, what=""):
    """GPU state [B,H,d+1,d] (S transposed, then z) against oracle S [B,H,d,d], z [B,H,d]."""
    d = S.shape[-1]
    Sg = state_gpu[..., :d, :].swapaxes(-1, -2)
    zg = state_gpu[..., d, :]
    for g, r, n in ((Sg, S, "S"), (zg, z, "z")):
        rms = np.sqrt((r ** 2).mean(axis=tuple(range(2, r.ndim)), keepdims=True))
        bound = rel * (np.abs(r) + rms)
        delta = np.abs(g - r)
        assert (delta <= bound).all(), f"{what} {n}: worst ratio {(delta / (bound + 1e-300)).max():.3f}"


def sample_rows(N, count, seed, tile=128):
    """Token rows to check at full size: ends, tile edges, and seeded random picks."""
    rng = np.random.default_rng(seed)
    fixed = [0, 1, tile - 1, tile, tile + 1, N // 2, N - tile - 1, N - tile, N - 2, N - 1]
    fixed = [r for r in fixed if 0 <= r < N]
    rnd = rng.integers(0, N, size=max(0, count - len(fixed)))
    return np.unique(np.concatenate([np.array(fixed, dtype=np.int64), rnd.astype(np.int64)]))


def read_golden(name):
    """Sections of a text fixture under tests/golden/: {'section': float64 array}, comment lines skipped."""
    import os

    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", name)
    out, key = {}, None
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("["):
            key = line.strip("[]")
            out[key] = []
        else:
            out[key].append([float(x) for x in line.split()])
    return {k: np.array(v, dtype=np.float64) for k, v in out.items()}
