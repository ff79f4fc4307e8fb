"""Parity at the full workload sizes, in the launch configuration bench.py times (kernel chosen
by the library, CUDA stream launches of the same entry point): outputs of sampled rows against
the oracle's dense definition restricted to those rows, plus properties that hold at any size."""
import numpy as np
import pytest
import torch

from paper_2512_24545_b200 import inputs, mdbf as M
from helpers import GpuLayer, TOL, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2512_24545_b200 import build
    build.build()
    assert torch.cuda.is_available()


def sampled_rows(d_out, n=48, seed=0):
    rng = np.random.default_rng(seed)
    rows = set(rng.choice(d_out, size=n, replace=False).tolist())
    rows.update([0, 1, 31, 32, 127, 128, d_out - 129, d_out - 33, d_out - 1])   # tile edges and the tail
    return np.array(sorted(r for r in rows if 0 <= r < d_out))


def check_rows(g, x, y, rows, tol):
    ref = g.oracle_forward_rows(x, rows)
    assert np.all(np.isfinite(y))
    assert rel_err(y[:, rows], ref) <= tol


@pytest.mark.parametrize("k", [1664, 2560])
def test_qproj_decode_full_size(k):
    spec = inputs.qproj(k)
    x = inputs.make_activations(spec, 1)
    with GpuLayer(spec, 1) as g:
        y = g.forward(x)
        assert M.mdbf_poll_status(g.h) == 0
        check_rows(g, x, y, sampled_rows(spec.d_out), TOL["bf16"])
        np.testing.assert_array_equal(y, g.forward(x))            # deterministic


@pytest.mark.parametrize("which,T", [("up", 1), ("up", 4), ("up", 16), ("down", 1), ("down", 4), ("down", 16)])
def test_mlp_small_batch_full_size(which, T):
    spec = inputs.mlp(which)
    x = inputs.make_activations(spec, T)
    with GpuLayer(spec, 16) as g:
        y = g.forward(x)
        assert M.mdbf_poll_status(g.h) == 0
        check_rows(g, x, y, sampled_rows(spec.d_out), TOL["bf16"])
        y0 = g.forward(x[:1])                                       # column independence
        assert rel_err(y0, y[:1]) <= 2 * TOL["bf16"]


@pytest.mark.parametrize("d_out,l,bpw", [(4096, 16, 1.0), (4096, 4, 1.5), (4096, 1, 1.0), (11008, 16, 1.5),
                                         (11008, 1, 1.5)])
def test_prefill_full_size(d_out, l, bpw):
    spec = inputs.prefill(d_out, l, bpw)
    T = 2048
    x = inputs.make_activations(spec, T)
    with GpuLayer(spec, T) as g:
        y = g.forward(x)
        assert M.mdbf_poll_status(g.h) == 0
        tok = np.array([0, 1, 15, 16, 255, 256, 1000, 2047])       # sampled tokens x sampled rows
        rows = sampled_rows(spec.d_out, n=24)
        ref = g.oracle_forward_rows(x[tok], rows)
        assert rel_err(y[np.ix_(tok, rows)], ref) <= TOL["bf16"]
        assert np.all(np.isfinite(y))
        # linearity at full size: a power-of-two scale is exact
        y2 = g.forward(2.0 * x[:64])
        np.testing.assert_array_equal(y2, 2.0 * g.forward(x[:64]))


@pytest.mark.parametrize("idx", [1, 4])      # k_proj 1024x8192 and gate 28672x8192
def test_block70b_layers_full_size(idx):
    spec = inputs.block70b()[idx]
    x = inputs.make_activations(spec, 1)
    with GpuLayer(spec, 1) as g:
        y = g.forward(x)
        assert M.mdbf_poll_status(g.h) == 0
        check_rows(g, x, y, sampled_rows(spec.d_out, n=16), TOL["bf16"])
