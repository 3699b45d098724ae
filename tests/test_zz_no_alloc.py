"""The workspace-free state entry point, `linattn_state_static_scratch`, against `linattn_state`.

It exists for callers that cannot allocate device memory when they need the state (fixed memory pools,
no allocator handed to a plug-in, threads that must stay off the allocator's lock); its scratch is an
array compiled into the library and shared by every call on a device.  The test calls it through the
C ABI twice in a row, with different problems, so that what the first call left in the shared array
would show up in the second, and checks each result against the ordinary entry point.  This file is
collected last on purpose: it must pass both on its own and after every other test has run.
"""
import ctypes

import numpy as np
import pytest

import synth
from parity_util import assert_state_close, to_dev, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def la():
    import torch

    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2509_24695_b200 as la

    la.load_library()
    return la


def _state_both_ways(la, shape, seed, dtype="bf16", kv=None):
    import torch

    B, N, H, d = shape
    k = to_dev(synth.gauss(shape, seed, 2, dtype=dtype) if kv is None else kv[0])
    v = to_dev(synth.gauss(shape, seed, 3, dtype=dtype) if kv is None else kv[1])
    ref = la.linattn_state(k, v)
    out = torch.full((B, H, d + 1, d), float("nan"), dtype=torch.float32, device="cuda")
    lib = la.load_library()
    desc = la._Desc(B, H, d, la._dtype_code(k), *k.stride()[:3])
    status = lib.linattn_state_static_scratch(ctypes.byref(desc), N, ctypes.c_void_p(k.data_ptr()),
                                              ctypes.c_void_p(v.data_ptr()), ctypes.c_void_p(out.data_ptr()),
                                              ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert status == 0, lib.linattn_status_string(status)
    torch.cuda.synchronize()
    assert la.static_scratch_status() == 0          # no bounded wait ran out in the launch just made
    # same kernel, same work split, same order of the partial sums: the two entry points agree bit for bit
    assert torch.equal(out, ref), "the built-in scratch changed the result"
    return to_f64(out), to_f64(ref)


def test_two_calls_in_a_row_match_linattn_state(la):
    # first a long sequence on the tensor-core path, then a shorter one with other values and another
    # head count: stale partial records or a stale control block would corrupt the second result
    for shape, seed in (((1, 5000, 20, 112), 4101), ((2, 777, 3, 112), 4102)):
        got, ref = _state_both_ways(la, shape, seed)
        d = shape[3]
        assert np.isfinite(got).all()
        assert_state_close(got, ref[..., :d, :].swapaxes(-1, -2), ref[..., d, :], 1e-5, f"static scratch {shape}")


def test_small_integers_match_the_oracle_bit_for_bit(la, orc):
    # inputs in {-2..2}: every partial sum is an integer below 2^24, so the fp32 state must equal the fp64
    # oracle's exactly, whatever the order of the sums -- twice in a row through the shared array
    for shape, seed in (((1, 3000, 5, 112), 4111), ((2, 1200, 3, 64), 4112)):
        k, v = synth.smallint(shape, seed, 2, 2), synth.smallint(shape, seed, 3, 2)
        got, _ = _state_both_ways(la, shape, seed, kv=(k, v))
        S, z = orc.state(k, v)
        d = shape[3]
        assert np.array_equal(got[..., :d, :].swapaxes(-1, -2), S) and np.array_equal(got[..., d, :], z), shape


def test_other_paths_and_repeat(la):
    # fp32 inputs (plain FMA kernels) and a packed head dim, then the first problem again
    got, ref = _state_both_ways(la, (1, 900, 2, 48), 4103, dtype="f32")
    assert_state_close(got, ref[..., :48, :].swapaxes(-1, -2), ref[..., 48, :], 1e-5, "static scratch fp32")
    got, ref = _state_both_ways(la, (1, 1500, 6, 64), 4104)
    assert_state_close(got, ref[..., :64, :].swapaxes(-1, -2), ref[..., 64, :], 1e-5, "static scratch d=64")
    got, ref = _state_both_ways(la, (1, 5000, 20, 112), 4101)
    assert_state_close(got, ref[..., :112, :].swapaxes(-1, -2), ref[..., 112, :], 1e-5, "static scratch again")


def test_too_large_is_refused_and_zero_tokens_is_an_empty_sum(la):
    import torch

    # 80 heads of dimension 112 need more split-N scratch than the built-in 16 MiB
    k = torch.zeros((1, 64, 80, 112), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((1, 80, 113, 112), dtype=torch.float32, device="cuda")
    with pytest.raises(la.LinAttnError) as e:
        la.linattn_state_static_scratch(k, k.clone(), out)
    assert e.value.status == -8
    # fp32 inputs keep one partial state per 512 tokens: 20 heads of dimension 112 fit up to 8192 tokens
    kf = torch.zeros((1, 8193, 20, 112), dtype=torch.float32, device="cuda")
    outf = torch.zeros((1, 20, 113, 112), dtype=torch.float32, device="cuda")
    with pytest.raises(la.LinAttnError) as e:
        la.linattn_state_static_scratch(kf, kf.clone(), outf)
    assert e.value.status == -8
    la.linattn_state_static_scratch(kf[:, :8192], kf[:, :8192].clone(), outf)
    k0 = torch.zeros((1, 0, 2, 112), dtype=torch.bfloat16, device="cuda")
    out0 = torch.ones((1, 2, 113, 112), dtype=torch.float32, device="cuda")
    la.linattn_state_static_scratch(k0, k0.clone(), out0)
    assert (out0 == 0).all()
