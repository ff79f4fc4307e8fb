"""CPU-only checks of the C-ABI library: it loads, exports every symbol the
header declares, its host-side packer is bit-exact against the oracle, and its
argument checking answers with status codes (no compute call needs a GPU)."""
import ctypes
import os
import re

import numpy as np
import pytest
import torch

from oracle import mdbf_oracle as orc
from paper_2512_24545_b200 import mdbf as M

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2512_24545_b200 import build
    build.build()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "mdbf.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mdbf_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = M.lib()
    names = declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(L, n), f"libmdbf.so does not export {n}"
    assert sorted(M.EXPORTS) == names, "binding and header disagree on the entry points"
    for n in names:
        assert hasattr(M, n) or n in ("mdbf_last_error", "mdbf_version")
    assert "sm_100a" in M.version()


def test_host_packer_bit_exact():
    rng = np.random.default_rng(5)
    for rows, cols in [(1, 1), (3, 31), (4, 32), (5, 33), (7, 200), (16, 256), (2, 1000)]:
        S = rng.choice(np.array([-1, 1], dtype=np.int8), size=(rows, cols))
        out = np.full((rows, (cols + 31) // 32), 0xDEADBEEF, dtype=np.uint32)
        M.mdbf_pack_signs(S, rows, cols, out, on_device=False)
        np.testing.assert_array_equal(out, orc.pack_signs(S))
        back = np.zeros((rows, cols), dtype=np.int8)
        M.mdbf_unpack_signs(out, rows, cols, back, on_device=False)
        np.testing.assert_array_equal(back, S)
        np.testing.assert_array_equal(orc.unpack_signs(out, cols), S)


def test_host_packer_patterns():
    for pat, word in [(np.ones(32), 0), (-np.ones(32), 0xFFFFFFFF),
                      (np.where(np.arange(32) % 2 == 0, 1, -1), 0xAAAAAAAA)]:
        S = pat.astype(np.int8)[None]
        out = np.zeros((1, 1), dtype=np.uint32)
        M.mdbf_pack_signs(S, 1, 32, out, on_device=False)
        assert int(out[0, 0]) == word
    for c in range(32):
        S = np.ones((1, 32), dtype=np.int8)
        S[0, c] = -1
        out = np.zeros((1, 1), dtype=np.uint32)
        M.mdbf_pack_signs(S, 1, 32, out, on_device=False)
        assert int(out[0, 0]) == 1 << c


def test_host_packer_rejects_bad_values_and_args():
    S = np.array([[1, 0, -1]], dtype=np.int8)
    out = np.zeros((1, 1), dtype=np.uint32)
    with pytest.raises(M.MdbfError) as e:
        M.mdbf_pack_signs(S, 1, 3, out, on_device=False)
    assert e.value.status == M.ERR_VALUE and "expected +1 or -1" in str(e.value)
    with pytest.raises(M.MdbfError) as e:
        M.mdbf_pack_signs(None, 1, 3, out, on_device=False)
    assert e.value.status == M.ERR_INVALID_ARG
    with pytest.raises(M.MdbfError) as e:
        M.mdbf_pack_signs(S, -1, 3, out, on_device=False)
    assert e.value.status == M.ERR_SHAPE
    M.mdbf_pack_signs(S, 0, 3, out, on_device=False)       # empty input is a no-op
    assert int(out[0, 0]) == 0


def test_handle_calls_reject_null_and_garbage():
    for fn, args in [(M.mdbf_destroy, ()), (M.mdbf_get_desc, ()), (M.mdbf_set_kernel, (0,)),
                     (M.mdbf_poll_status, ()), (M.mdbf_last_launch_count, ()), (M.mdbf_last_kernel, ())]:
        with pytest.raises(M.MdbfError) as e:
            fn(0, *args)
        assert e.value.status == M.ERR_INVALID_ARG
    junk = (ctypes.c_uint32 * 64)()
    with pytest.raises(M.MdbfError) as e:
        M.mdbf_linear_forward(ctypes.addressof(junk), 1, 1, 1, M.BF16)
    assert e.value.status == M.ERR_INVALID_ARG and "invalid handle" in str(e.value)


def test_pack_argument_checks_need_no_gpu():
    S = np.ones((4, 4), dtype=np.int8)
    F = np.ones((4, 1), dtype=np.float32)
    with pytest.raises(M.MdbfError) as e:
        M.mdbf_pack(4, 4, 4, 0, M.F16, 1, S, S, F, F, F, F)          # l = 0
    assert e.value.status == M.ERR_SHAPE
    with pytest.raises(M.MdbfError) as e:
        M.mdbf_pack(4, 4, 4, 1, 7, 1, S, S, F, F, F, F)              # bad dtype
    assert e.value.status == M.ERR_DTYPE
    with pytest.raises(M.MdbfError) as e:
        M.mdbf_pack(4, 4, 4, 1, M.F16, 1, None, S, F, F, F, F)
    assert e.value.status == M.ERR_INVALID_ARG


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device answer")
def test_no_cpu_fallback_without_a_device():
    """Without a CUDA device the compute entry points fail loudly with MDBF_ERR_ARCH."""
    S = np.ones((4, 4), dtype=np.int8)
    F = np.ones((4, 1), dtype=np.float32)
    with pytest.raises(M.MdbfError) as e:
        M.mdbf_pack(4, 4, 4, 1, M.F16, 1, S, S, F, F, F, F)
    assert e.value.status == M.ERR_ARCH and "CUDA device" in str(e.value)
    out = np.zeros((4, 1), dtype=np.uint32)
    with pytest.raises(M.MdbfError) as e:
        M.mdbf_pack_signs(S, 4, 4, out, on_device=True)
    assert e.value.status == M.ERR_ARCH


def test_msvid_workspace_size_is_a_host_computation():
    """No device needed: the size grows with the shape and the envelope rank, bad shapes are refused."""
    a = M.mdbf_msvid_workspace_bytes(1024, 768, 4)
    b = M.mdbf_msvid_workspace_bytes(1024, 768, 16)
    c = M.mdbf_msvid_workspace_bytes(4096, 768, 16)
    assert 0 < a < b < c and a % 256 == 0
    assert M.mdbf_msvid_workspace_bytes(1024, 768, 5) == M.mdbf_msvid_workspace_bytes(1024, 768, 8)   # rank padded to a power of two
    for bad in ((0, 8, 1), (8, 0, 1), (8, 8, 0), (8, 8, 9), (8, 8, 33)):
        with pytest.raises(M.MdbfError) as e:
            M.mdbf_msvid_workspace_bytes(*bad)
        assert e.value.status == M.ERR_SHAPE
