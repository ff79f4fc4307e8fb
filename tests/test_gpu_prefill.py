"""Parity of the large-T (tcgen05) kernel with the CPU oracle on small shapes
that still span several 128-row tiles, several K blocks and ragged tails."""
import numpy as np
import pytest
import torch

from oracle import mdbf_oracle as orc
from paper_2512_24545_b200 import inputs, mdbf as M
from helpers import check_parity, GpuLayer, rel_err, TOL

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2512_24545_b200 import build
    build.build()
    assert torch.cuda.is_available()


def spec_of(d_out, d_in, k, l, **kw):
    return inputs.scaled(inputs.qproj(1664), name="pf", d_out=d_out, d_in=d_in, k=k, l=l, outliers=False, **kw)


@pytest.mark.parametrize("l,T", [(16, 16), (16, 48), (16, 5), (4, 64), (4, 100), (1, 256), (1, 300),
                                 (3, 40), (8, 33), (20, 9), (32, 11)])
def test_prefill_kernel_small_shapes(l, T):
    spec = spec_of(384, 576, 256, l)
    x = inputs.make_activations(spec, T)
    with GpuLayer(spec, T) as g:
        ref = g.oracle_forward(x)
        y = g.forward(x, kernel=M.KERNEL_PREFILL)
        assert M.mdbf_poll_status(g.h) == 0
        check_parity(g, x, y, ref, roundings=3)
        _, z_ref = orc.forward_staged(*g.oracle_args(), x.T.astype(np.float64))
        assert rel_err(g.intermediate(T), z_ref.T) <= TOL["bf16"]


@pytest.mark.parametrize("shape", [(1, 1, 1, 1), (100, 70, 50, 2), (129, 65, 130, 16), (300, 1000, 260, 5)])
def test_prefill_kernel_ragged_shapes(shape):
    d_out, d_in, k, l = shape
    spec = spec_of(d_out, d_in, k, l)
    x = inputs.make_activations(spec, 19)
    with GpuLayer(spec, 19) as g:
        y = g.forward(x, kernel=M.KERNEL_PREFILL)
        assert M.mdbf_poll_status(g.h) == 0
        # 5e-3 bounds the Frobenius (RMS) error of many independently rounded terms; a layer with a few terms per
        # output has nothing to average, so there the per-element bound (three bf16 roundings: scaled x, scaled z, y)
        # is the assertion
        check_parity(g, x, y, roundings=3, averaging=k >= 8)


def test_prefill_agrees_with_small_T_kernel_and_auto_dispatch():
    spec = spec_of(256, 512, 256, 16, env_dtype="bf16")
    x = inputs.make_activations(spec, 4)
    with GpuLayer(spec, 64) as g:
        ref = g.oracle_forward(x)
        y_pf = g.forward(x, kernel=M.KERNEL_PREFILL)
        y_alu = g.forward(x, kernel=M.KERNEL_ALU)
        assert rel_err(y_pf, ref) <= TOL["bf16"] and rel_err(y_alu, ref) <= TOL["bf16"]
        assert rel_err(y_pf, y_alu) <= 2 * TOL["bf16"]
        x64 = inputs.make_activations(spec, 64)
        y_auto = g.forward(x64)                       # T >= 2 -> materialised-order kernel
        assert M.mdbf_last_kernel(g.h) == M.KERNEL_MAT
        assert rel_err(y_auto, g.oracle_forward(x64)) <= TOL["bf16"]
        np.testing.assert_array_equal(y_auto, g.forward(x64, kernel=M.KERNEL_MAT))


def test_envelope_rank_above_32_takes_the_fp32_path():
    spec = spec_of(96, 160, 64, 40)
    x = inputs.make_activations(spec, 6)
    with GpuLayer(spec, 6) as g:
        assert rel_err(g.forward(x), g.oracle_forward(x)) <= TOL["bf16"]       # AUTO -> ALU kernel
        with pytest.raises(M.MdbfError) as e:
            g.forward(x, kernel=M.KERNEL_PREFILL)
        assert e.value.status == M.ERR_DTYPE
