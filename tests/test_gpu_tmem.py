"""Parity of the one-token tcgen05 kernel with a bf16 operand in TMEM (sign XOR-ed into the activation, cluster
split of the reduction) with the CPU oracle: shapes spanning several 128-row blocks, several K blocks per cluster
rank, ragged tails, every envelope-rank bucket and both 16-bit envelope types."""
import numpy as np
import pytest
import torch

from oracle import mdbf_oracle as orc
from paper_2512_24545_b200 import inputs, mdbf as M
from helpers import GpuLayer, TOL, check_parity, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2512_24545_b200 import build
    build.build()
    assert torch.cuda.is_available()


def spec_of(d_out, d_in, k, l, **kw):
    return inputs.scaled(inputs.qproj(1664), name="tm", d_out=d_out, d_in=d_in, k=k, l=l, **kw)


def test_tmem_kernel_smallest_case():
    spec = spec_of(128, 64, 64, 16, outliers=False)
    x = inputs.make_activations(spec, 1)
    with GpuLayer(spec, 1) as g:
        y = g.forward(x, kernel=M.KERNEL_TMEM)
        assert M.mdbf_poll_status(g.h) == 0
        check_parity(g, x, y)


@pytest.mark.parametrize("l", [1, 2, 3, 4, 8, 12, 16, 24, 32])
@pytest.mark.parametrize("env", ["f16", "bf16"])
def test_one_token_kernel(l, env):
    """The activation is folded into the TMEM operand (sign XOR-ed into the bf16 activation pair)."""
    spec = spec_of(419, 1000, 700, l, env_dtype=env)
    x = inputs.make_activations(spec, 1)
    with GpuLayer(spec, 4) as g:
        ref = g.oracle_forward(x)
        y = g.forward(x, kernel=M.KERNEL_TMEM)
        assert M.mdbf_poll_status(g.h) == 0
        check_parity(g, x, y, ref)
        _, z_ref = orc.forward_staged(*g.oracle_args(), x.T.astype(np.float64))
        assert rel_err(g.intermediate(1), z_ref.T) <= TOL["bf16"]
        np.testing.assert_array_equal(y, g.forward(x, kernel=M.KERNEL_TMEM))      # deterministic
        check_parity(g, x, g.forward(x), ref)                                      # whatever AUTO picks
        x4 = inputs.make_activations(spec, 4)                     # same layer, wider batch: another kernel, same layer
        y4 = g.forward(x4)
        check_parity(g, x4, y4)
        assert rel_err(g.forward(x4[:1], kernel=M.KERNEL_TMEM), y4[:1]) <= 2 * TOL["bf16"]


@pytest.mark.parametrize("shape", [(1, 1, 1, 1), (31, 127, 33, 2), (129, 1025, 257, 9), (1000, 2100, 1300, 16),
                                   (256, 4096, 512, 16), (2048, 192, 3000, 16)])
def test_tmem_kernel_edge_shapes(shape):
    d_out, d_in, k, l = shape
    spec = spec_of(d_out, d_in, k, l)
    x = inputs.make_activations(spec, 1)
    with GpuLayer(spec, 1) as g:
        y = g.forward(x, kernel=M.KERNEL_TMEM)
        assert M.mdbf_poll_status(g.h) == 0
        check_parity(g, x, y, averaging=k >= 8)                 # a layer with a few terms: the per-element bound


def test_tmem_kernel_takes_one_token_only():
    spec = spec_of(128, 128, 128, 16)
    x = inputs.make_activations(spec, 2)
    with GpuLayer(spec, 2) as g:
        with pytest.raises(M.MdbfError) as e:
            g.forward(x, kernel=M.KERNEL_TMEM)
        assert e.value.status == M.ERR_SHAPE
        check_parity(g, x, g.forward(x))                         # AUTO -> materialised-envelope kernel
        with pytest.raises(M.MdbfError) as e:
            M.mdbf_set_kernel(g.h, 2)                            # the retired selector
        assert e.value.status == M.ERR_INVALID_ARG


def test_bounded_wait_times_out_and_the_context_survives():
    """A device-side wait that can never complete gives up after its time limit, reports
    MDBF_ERR_TIMEOUT through the status word, and leaves the context usable."""
    import time
    spec = spec_of(128, 128, 128, 16)
    x = inputs.make_activations(spec, 1)
    with GpuLayer(spec, 1) as g:
        assert M.mdbf_poll_status(g.h) == 0
        t0 = time.perf_counter()
        M.mdbf_selftest_wait_timeout(g.h, torch.cuda.current_stream().cuda_stream)
        status = M.mdbf_poll_status(g.h)                           # synchronises
        dt = time.perf_counter() - t0
        assert status == M.ERR_TIMEOUT
        assert 0.5 < dt < 10.0
        assert M.mdbf_poll_status(g.h) == 0                        # reading cleared it
        assert rel_err(g.forward(x), g.oracle_forward(x)) <= TOL["bf16"]       # still works
        assert M.mdbf_poll_status(g.h) == 0
