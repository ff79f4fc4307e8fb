"""Parity at the full workload sizes, in the launch configuration bench.py times (kernel chosen
by the library, CUDA stream launches of the same entry point): outputs of sampled rows against
the oracle's dense definition restricted to those rows, plus properties that hold at any size."""
import numpy as np
import pytest
import torch

from paper_2512_24545_b200 import inputs, mdbf as M
from helpers import GpuLayer, TOL, magnitude_bound, rel_err

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


PREFILL_POINTS = [(d_out, l, bpw) for d_out in (4096, 11008) for l in (1, 4, 16) for bpw in (1.0, 1.5)]


def check_tokens_rows(g, x, y, rows, tok):
    ref = g.oracle_forward_rows(x[tok], rows)
    assert np.all(np.isfinite(y))
    got = y[np.ix_(tok, rows)]
    assert rel_err(got, ref) <= TOL["bf16"]
    # every sampled element on its own (no token or row hides in the norm): four bf16 roundings at most on any path
    bound = magnitude_bound(g, x[tok], rows)
    assert np.all(np.abs(got - ref) <= 5 * 2.0 ** -8 * bound)


@pytest.mark.parametrize("d_out,l,bpw", PREFILL_POINTS)
def test_prefill_full_size(d_out, l, bpw):
    """All twelve points of the prefill sweep (both shapes, l in {1, 4, 16}, ~1.0 and ~1.5 bpw) at T = 2048
    under the library's own choice of kernel."""
    spec = inputs.prefill(d_out, l, bpw)
    T = 2048
    x = inputs.make_activations(spec, T)
    with GpuLayer(spec, T) as g:
        y = g.forward(x)
        assert M.mdbf_poll_status(g.h) == 0
        tok = np.array([0, 1, 15, 16, 255, 256, 1000, 2047])       # sampled tokens x sampled rows
        check_tokens_rows(g, x, y, sampled_rows(spec.d_out, n=24), tok)
        # linearity at full size: a power-of-two scale is exact
        y2 = g.forward(2.0 * x[:64])
        np.testing.assert_array_equal(y2, 2.0 * g.forward(x[:64]))


@pytest.mark.parametrize("d_out,l,bpw", [(4096, 16, 1.0), (11008, 1, 1.5), (4096, 4, 1.5)])
def test_prefill_full_size_expanded_order(d_out, l, bpw):
    """The expanded-order kernel (pre-scale, l sign GEMMs of width l T, mode contraction in the epilogue) at T = 2048."""
    spec = inputs.prefill(d_out, l, bpw)
    T = 2048
    x = inputs.make_activations(spec, T)
    with GpuLayer(spec, T) as g:
        y = g.forward(x, kernel=M.KERNEL_PREFILL)
        assert M.mdbf_poll_status(g.h) == 0
        assert M.mdbf_last_kernel(g.h) == M.KERNEL_PREFILL
        tok = np.array([0, 1, 15, 16, 255, 256, 1000, 2047])
        check_tokens_rows(g, x, y, sampled_rows(spec.d_out, n=24), tok)


@pytest.mark.parametrize("idx", range(7))      # q, k, v, o, gate, up, down of the 70B-class block
def test_block70b_layers_full_size_one_token(idx):
    spec = inputs.block70b()[idx]
    x = inputs.make_activations(spec, 1)
    with GpuLayer(spec, 1) as g:
        y = g.forward(x)
        assert M.mdbf_poll_status(g.h) == 0
        check_rows(g, x, y, sampled_rows(spec.d_out, n=16), TOL["bf16"])
        y8 = g.forward(x, kernel=M.KERNEL_I8)                       # both one-token kernels at full size
        check_rows(g, x, y8, sampled_rows(spec.d_out, n=16), TOL["bf16"])


def test_block70b_siblings_full_size_one_token():
    """q/k/v and gate/up through the sibling entry point, as bench.py runs the block."""
    specs = inputs.block70b()
    for group in ([0, 1, 2], [4, 5]):
        layers = [GpuLayer(specs[i], 1) for i in group]
        try:
            x = inputs.make_activations(specs[group[0]], 1)
            xd = torch.from_numpy(x).to(torch.bfloat16).cuda()
            ys = [torch.full((1, specs[i].d_out), float("nan"), dtype=torch.bfloat16, device="cuda") for i in group]
            M.mdbf_linear_forward_siblings([g.h for g in layers], xd.data_ptr(), [y.data_ptr() for y in ys], 1, M.BF16,
                                           torch.cuda.current_stream().cuda_stream)
            torch.cuda.synchronize()
            for g, y in zip(layers, ys):
                assert M.mdbf_poll_status(g.h) == 0
                check_rows(g, x, y.to(torch.float32).cpu().numpy(), sampled_rows(g.spec.d_out, n=12), TOL["bf16"])
        finally:
            for g in layers:
                g.close()


@pytest.mark.parametrize("idx", range(7))
def test_block70b_layers_full_size_2048_tokens(idx):
    spec = inputs.block70b()[idx]
    T = 2048
    x = inputs.make_activations(spec, T)
    with GpuLayer(spec, T) as g:
        y = g.forward(x)
        assert M.mdbf_poll_status(g.h) == 0
        tok = np.array([0, 255, 256, 1033, 2047])
        check_tokens_rows(g, x, y, sampled_rows(spec.d_out, n=8), tok)


SECOND_SEED = 90001


@pytest.mark.parametrize("case", ["qproj1664", "qproj2560", "up_T1", "down_T16", "gate_T1", "down70b_T1", "prefill4096", "prefill11008"])
def test_second_seed_with_outlier_channels(case):
    """The margin under the 5e-3 bound does not hinge on the seeds of the workload table: every config once more with
    other seeds, and with the 1 % outlier channels (x20) switched on for the prefill shapes as well."""
    if case.startswith("qproj"):
        spec, T = inputs.qproj(int(case[5:])), 1
    elif case == "up_T1":
        spec, T = inputs.mlp("up"), 1
    elif case == "down_T16":
        spec, T = inputs.mlp("down"), 16
    elif case == "gate_T1":
        spec, T = inputs.block70b()[4], 1
    elif case == "down70b_T1":
        spec, T = inputs.block70b()[6], 1
    elif case == "prefill4096":
        spec, T = inputs.prefill(4096, 16, 1.0), 2048
    else:
        spec, T = inputs.prefill(11008, 4, 1.5), 2048
    spec = inputs.scaled(spec, seed=spec.seed + SECOND_SEED, outliers=True)
    x = inputs.make_activations(spec, T)
    rows = sampled_rows(spec.d_out, n=16, seed=1)
    tok = np.unique(np.array([0, T // 3, T - 1]))
    with GpuLayer(spec, T) as g:
        kernels = [M.KERNEL_AUTO] + ([M.KERNEL_I8, M.KERNEL_TMEM] if T == 1 else [])
        for kernel in kernels:
            y = g.forward(x, kernel=kernel)
            check_tokens_rows(g, x, y, rows, tok)
