"""The C-ABI shared library: it builds for sm_100a, loads without a GPU, exports every symbol the
public header declares, and its host-side validation answers without touching a device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2509_24695_b200 import build, load_library

    build.build()
    return load_library()


def declared_symbols():
    import glob

    text = "".join(open(h).read() for h in sorted(glob.glob(os.path.join(ROOT, "include", "*.h"))))
    return sorted(set(re.findall(r"LINATTN_API\s+[\w\s\*]+?\b((?:linattn|blocklin|tconv)_\w+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = declared_symbols()
    assert {"linattn_forward", "linattn_state", "linattn_apply", "blocklin_cache_init", "blocklin_cache_reset",
            "blocklin_step", "blocklin_prefill", "tconv_forward", "tconv_block_step", "tconv_prefill",
            "tconv_cache_bytes", "tconv_cache_reset"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in linattn.h but not exported"


def test_header_compiles_as_plain_c(tmp_path):
    import subprocess

    src = tmp_path / "t.c"
    src.write_text('#include "linattn.h"\n#include "tconv.h"\n'
                   'int main(void){ linattn_desc d; tconv_desc c; (void)d; (void)c; return LINATTN_OK; }\n')
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), "-c", str(src),
                           "-o", str(tmp_path / "t.o")])


def test_sizes_and_validation_without_gpu(lib):
    import paper_2509_24695_b200 as la

    # Table 1: the cache is O(d^2) per head and nothing else
    assert la.state_bytes(1, 20, 112) == 20 * (112 * 112 + 112) * 4 == 1012480
    assert la.state_bytes(2, 20, 112) == 2024960
    w1 = la.workspace_bytes(1, 20, 112, 32760)
    assert w1 >= la.WORKSPACE_CTRL_BYTES + 1012480 and w1 % 256 == 0
    assert la.workspace_bytes(1, 20, 112, 0) >= la.WORKSPACE_CTRL_BYTES
    for args, status in [((0, 20, 112, 10), -1), ((1, 20, 0, 10), -1), ((1, 20, 129, 10), -2), ((1, 20, 112, -1), -1)]:
        with pytest.raises(la.LinAttnError) as e:
            la.workspace_bytes(*args)
        assert e.value.status == status
    assert lib.linattn_status_string(0) == b"ok"
    assert b"workspace" in lib.linattn_status_string(-4)
    # null pointers are rejected before any launch
    d = la._Desc(1, 2, 112, 0, 0, 0, 0)
    assert lib.linattn_forward(ctypes.byref(d), 8, None, None, None, None, 1e-6, None, 0, None) == -1
    assert lib.linattn_forward(None, 8, None, None, None, None, 1e-6, None, 0, None) == -1
    assert lib.blocklin_step(None, 8, None, None, None, None, None) == -7
    assert lib.blocklin_cache_reset(None, None) == -7
    assert lib.blocklin_cache_destroy(None) == -7
    sb, wb = ctypes.c_size_t(), ctypes.c_size_t()
    assert lib.blocklin_cache_bytes(ctypes.byref(d), 4680, ctypes.byref(sb), ctypes.byref(wb)) == 0
    assert sb.value == 2 * (112 * 112 + 112) * 4
    h = ctypes.c_void_p()
    assert lib.blocklin_cache_init(ctypes.byref(h), ctypes.byref(d), 1e-6, None, sb.value, None, wb.value, None) == -1
    assert not h.value


def test_product_package_does_not_touch_the_oracle():
    """The oracle and the seeded input generator are test infrastructure: nothing under the package may import
    or load them (and neither of the two imports the other or the package)."""
    for mod, banned in (("oracle", ("import synth", "paper_2509_24695_b200", "libsynth")),
                        ("synth", ("import oracle", "from oracle", "paper_2509_24695_b200", "liblinattn"))):
        for dirpath, _, files in os.walk(os.path.join(ROOT, mod)):
            for f in files:
                if f.endswith((".py", ".c", ".h")):
                    text = open(os.path.join(dirpath, f)).read()
                    assert not any(b in text for b in banned), (mod, f)
    pkg = os.path.join(ROOT, "paper_2509_24695_b200")
    for dirpath, _, files in os.walk(pkg):
        if "_build" in dirpath:
            continue
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".c", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text and "liblinattn_oracle" not in text, f
                assert "import synth" not in text and "libsynth" not in text, f


def test_tconv_sizes_and_validation_without_gpu(lib):
    import paper_2509_24695_b200 as la

    nbytes = ctypes.c_size_t()
    d = la._ConvDesc(2, 30 * 52, 2240, 0, 0, 0)
    assert lib.tconv_cache_bytes(ctypes.byref(d), ctypes.byref(nbytes)) == 0
    assert nbytes.value == 2 * 30 * 52 * 2240 * 2            # one frame per batch entry, nothing per block
    d32 = la._ConvDesc(1, 10, 16, 1, 0, 0)
    assert lib.tconv_cache_bytes(ctypes.byref(d32), ctypes.byref(nbytes)) == 0 and nbytes.value == 10 * 16 * 4
    assert lib.tconv_cache_bytes(ctypes.byref(la._ConvDesc(1, 10, 12, 0, 0, 0)), ctypes.byref(nbytes)) == -2
    assert lib.tconv_cache_bytes(ctypes.byref(la._ConvDesc(0, 10, 16, 0, 0, 0)), ctypes.byref(nbytes)) == -1
    assert lib.tconv_cache_bytes(None, ctypes.byref(nbytes)) == -1
    # null tensors and negative sizes are rejected before any launch
    assert lib.tconv_forward(ctypes.byref(d), 3, None, None, None, None) == -1
    assert lib.tconv_forward(ctypes.byref(d), -1, None, None, None, None) == -1
    assert lib.tconv_block_step(ctypes.byref(d), 3, None, None, None, None, 1, None) == -1
    assert lib.tconv_prefill(ctypes.byref(d), -1, 3, None, None, None, None, None) == -1


def test_prefill_workspace_size_without_gpu(lib):
    """Room for taking all blocks of a prefill together: never less than what single steps need, grows with the
    number of blocks (one more set of per-block states and records each), refuses what the grid cannot index."""
    import paper_2509_24695_b200 as la

    d = la._Desc(1, 20, 112, 0, 0, 0, 0)
    step_state, step_ws, pre = ctypes.c_size_t(), ctypes.c_size_t(), ctypes.c_size_t()
    assert lib.blocklin_cache_bytes(ctypes.byref(d), 4680, ctypes.byref(step_state), ctypes.byref(step_ws)) == 0
    assert lib.blocklin_prefill_workspace_bytes(ctypes.byref(d), 1, 4680, ctypes.byref(pre)) == 0
    one = pre.value
    assert lib.blocklin_prefill_workspace_bytes(ctypes.byref(d), 7, 4680, ctypes.byref(pre)) == 0
    assert pre.value > one and pre.value >= 7 * step_state.value and pre.value % 256 == 0
    assert lib.blocklin_prefill_workspace_bytes(ctypes.byref(d), 4000, 4680, ctypes.byref(pre)) == -2   # 80 000 units
    assert lib.blocklin_prefill_workspace_bytes(ctypes.byref(d), 0, 4680, ctypes.byref(pre)) == -1
    assert lib.blocklin_prefill_workspace_bytes(ctypes.byref(d), 7, 4680, None) == -1
