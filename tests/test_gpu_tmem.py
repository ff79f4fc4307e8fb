"""Parity of the small-T tcgen05 kernel (sign operand in TMEM, cluster split of the reduction)
with the CPU oracle: shapes spanning several 128-row blocks, several K blocks per cluster rank,
ragged tails, every envelope-rank bucket and both 16-bit envelope types."""
import numpy as np
import pytest
import torch

from oracle import mdbf_oracle as orc
from paper_2512_24545_b200 import inputs, mdbf as M
from helpers import GpuLayer, TOL, rel_err

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
        assert rel_err(y, g.oracle_forward(x)) <= TOL["bf16"]


@pytest.mark.parametrize("l,T", [(16, 1), (16, 2), (16, 3), (16, 4), (1, 1), (1, 16), (2, 5), (3, 7), (4, 16),
                                 (8, 8), (12, 2), (24, 2), (32, 1)])
def test_tmem_kernel_small_shapes(l, T):
    spec = spec_of(352, 544, 320, l)
    x = inputs.make_activations(spec, T)
    with GpuLayer(spec, T) as g:
        ref = g.oracle_forward(x)
        y = g.forward(x, kernel=M.KERNEL_TMEM)
        assert M.mdbf_poll_status(g.h) == 0
        assert np.all(np.isfinite(y))
        assert rel_err(y, ref) <= TOL["bf16"]
        _, z_ref = orc.forward_staged(*g.oracle_args(), x.T.astype(np.float64))
        assert rel_err(g.intermediate(T), z_ref.T) <= TOL["bf16"]
        np.testing.assert_array_equal(y, g.forward(x, kernel=M.KERNEL_TMEM))      # deterministic
        assert rel_err(g.forward(x), ref) <= TOL["bf16"]                           # whatever AUTO picks


@pytest.mark.parametrize("l", [1, 2, 3, 4, 8, 12, 16, 24, 32])
@pytest.mark.parametrize("env", ["f16", "bf16"])
def test_one_token_kernel(l, env):
    """T = 1 takes the variant with the activation folded into the TMEM operand."""
    spec = spec_of(419, 1000, 700, l, env_dtype=env)
    x = inputs.make_activations(spec, 1)
    with GpuLayer(spec, 4) as g:
        ref = g.oracle_forward(x)
        y = g.forward(x, kernel=M.KERNEL_TMEM)
        assert M.mdbf_poll_status(g.h) == 0
        assert rel_err(y, ref) <= TOL["bf16"]
        _, z_ref = orc.forward_staged(*g.oracle_args(), x.T.astype(np.float64))
        assert rel_err(g.intermediate(1), z_ref.T) <= TOL["bf16"]
        x4 = inputs.make_activations(spec, 4)                     # same layer, wider batch: the B-scaled variant
        y4 = g.forward(x4, kernel=M.KERNEL_TMEM) if 4 * g.spec.l <= 64 and l in (1, 2, 4, 8, 16) else g.forward(x4)
        assert rel_err(y4, g.oracle_forward(x4)) <= TOL["bf16"]
        assert rel_err(g.forward(x4[:1], kernel=M.KERNEL_TMEM), y4[:1]) <= 2 * TOL["bf16"]


@pytest.mark.parametrize("shape", [(1, 1, 1, 1), (31, 127, 33, 2), (129, 1025, 257, 9), (1000, 2100, 1300, 16),
                                   (256, 4096, 512, 16), (2048, 192, 3000, 16)])
def test_tmem_kernel_edge_shapes(shape):
    d_out, d_in, k, l = shape
    spec = spec_of(d_out, d_in, k, l)
    x = inputs.make_activations(spec, 2)
    with GpuLayer(spec, 2) as g:
        y = g.forward(x, kernel=M.KERNEL_TMEM)
        assert M.mdbf_poll_status(g.h) == 0
        tol = 4 * 2.0 ** -9 if k == 1 else TOL["bf16"]           # a one-term layer has nothing to average
        assert rel_err(y, g.oracle_forward(x)) <= tol


def test_tmem_kernel_bf16_envelopes_and_cross_check():
    spec = spec_of(384, 512, 256, 16, env_dtype="bf16")
    x = inputs.make_activations(spec, 4)
    with GpuLayer(spec, 64) as g:
        ref = g.oracle_forward(x)
        y_tm = g.forward(x, kernel=M.KERNEL_TMEM)
        y_dec = g.forward(x, kernel=M.KERNEL_DECODE)
        y_pf = g.forward(x, kernel=M.KERNEL_PREFILL)
        for y in (y_tm, y_dec, y_pf):
            assert rel_err(y, ref) <= TOL["bf16"]
        assert rel_err(y_tm, y_pf) <= 2 * TOL["bf16"]
        for t in (0, 2):                                         # column independence inside one kernel variant
            assert rel_err(g.forward(x[t:t + 2], kernel=M.KERNEL_TMEM), y_tm[t:t + 2]) <= 1e-6
        for t in range(4):                                       # one token takes another variant: same within rounding
            assert rel_err(g.forward(x[t:t + 1], kernel=M.KERNEL_TMEM), y_tm[t:t + 1]) <= 2 * TOL["bf16"]


def test_tmem_kernel_rejects_wide_batches():
    spec = spec_of(128, 128, 128, 16)
    x = inputs.make_activations(spec, 8)
    with GpuLayer(spec, 8) as g:
        with pytest.raises(M.MdbfError) as e:
            g.forward(x, kernel=M.KERNEL_TMEM)                   # 16 modes x 8 tokens > 64 columns
        assert e.value.status == M.ERR_SHAPE
        assert rel_err(g.forward(x), g.oracle_forward(x)) <= TOL["bf16"]      # AUTO -> large-T kernel


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
