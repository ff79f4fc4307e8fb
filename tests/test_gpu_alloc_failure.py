"""Allocation failures injected on the host (mdbf_debug_fail_alloc makes the n-th device allocation of the library
return an error without touching the device): every call that allocates either completes or fails with
MDBF_ERR_ALLOC, frees what it took, publishes nothing half-built, and leaves the handle as usable as before.  No
GPU fault is involved: a failed build never reaches a kernel."""
import numpy as np
import pytest
import torch

from paper_2512_24545_b200 import inputs, mdbf as M
from helpers import GpuLayer, rel_err, TOL

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2512_24545_b200 import build
    build.build()
    assert torch.cuda.is_available()
    yield
    M.mdbf_debug_fail_alloc(0)


SPEC = inputs.scaled(inputs.qproj(1664), name="allocfail", d_out=384, d_in=512, k=256, l=16, outliers=False)


def free_bytes():
    torch.cuda.synchronize()
    return torch.cuda.mem_get_info()[0]


def pack_args(spec):
    lay = inputs.make_layer(spec)
    return [np.ascontiguousarray(lay[n]) for n in ("S_A", "S_B", "U_A", "V_A", "U_B", "V_B")]


@pytest.mark.parametrize("spec,max_T", [(SPEC, 64), (SPEC, 1), (inputs.tiny(), 8)])
def test_pack_fails_cleanly_at_every_allocation(spec, max_T):
    args = pack_args(spec)
    h = M.mdbf_pack(spec.d_out, spec.d_in, spec.k, spec.l, M.DTYPES[spec.env_dtype], max_T, *args)   # warm: contexts, modules
    M.mdbf_destroy(h)
    before = free_bytes()
    failures = 0
    for nth in range(1, 200):
        M.mdbf_debug_fail_alloc(nth)
        try:
            h = M.mdbf_pack(spec.d_out, spec.d_in, spec.k, spec.l, M.DTYPES[spec.env_dtype], max_T, *args)
        except M.MdbfError as e:
            assert e.status == M.ERR_ALLOC
            failures += 1
            assert free_bytes() == before                      # everything the failed call took is back
            continue
        finally:
            M.mdbf_debug_fail_alloc(0)
        M.mdbf_destroy(h)                                      # nth is beyond the allocations of a pack: it went through
        break
    else:
        pytest.fail("mdbf_pack never succeeded")
    assert failures >= 8                                       # signs, envelopes, layouts, scratch, status: all were hit
    assert free_bytes() == before


def test_lazy_scratch_fails_cleanly_and_the_handle_stays_usable():
    x = inputs.make_activations(SPEC, 8)
    with GpuLayer(SPEC, 64) as g:
        ref = g.oracle_forward(x)
        before = free_bytes()
        failures = 0
        for nth in range(1, 50):
            M.mdbf_debug_fail_alloc(nth)
            try:
                M.mdbf_set_kernel(g.h, M.KERNEL_PREFILL)       # builds the K-blocked words, the transposed V_B, the pre-scaled operands
            except M.MdbfError as e:
                assert e.status == M.ERR_ALLOC
                failures += 1
                M.mdbf_debug_fail_alloc(0)
                # nothing half-built was published: the default path still serves the handle, and the expanded order
                # is refused with a status instead of running on missing buffers
                assert rel_err(g.forward(x), ref) <= TOL["bf16"]
                continue
            finally:
                M.mdbf_debug_fail_alloc(0)
            break
        else:
            pytest.fail("mdbf_set_kernel never succeeded")
        assert failures >= 3
        assert rel_err(g.forward(x, kernel=M.KERNEL_PREFILL), ref) <= TOL["bf16"]
        assert free_bytes() < before                            # the scratch is there now


def test_host_staging_fails_cleanly():
    x = inputs.make_activations(SPEC, 4)
    with GpuLayer(SPEC, 4) as g:
        xh = torch.from_numpy(x).to(torch.bfloat16).pin_memory()
        yh = torch.zeros((4, SPEC.d_out), dtype=torch.bfloat16).pin_memory()
        st = torch.cuda.current_stream().cuda_stream
        for nth in (1, 2):
            before = free_bytes()
            M.mdbf_debug_fail_alloc(nth)
            with pytest.raises(M.MdbfError) as e:
                M.mdbf_prepare_host_staging(g.h)
            M.mdbf_debug_fail_alloc(0)
            assert e.value.status == M.ERR_ALLOC
            assert free_bytes() == before
            with pytest.raises(M.MdbfError) as e:               # still no staging: the host entry point says so, it never allocates
                M.mdbf_linear_forward_host(g.h, xh.data_ptr(), yh.data_ptr(), 4, M.BF16, st)
            assert e.value.status == M.ERR_INVALID_ARG
        M.mdbf_prepare_host_staging(g.h)
        M.mdbf_linear_forward_host(g.h, xh.data_ptr(), yh.data_ptr(), 4, M.BF16, st)
        np.testing.assert_array_equal(yh.to(torch.float32).numpy(), g.forward(x))
