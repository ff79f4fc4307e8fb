"""Sum of P layers on one input (residual compensation, Eq. dbf-residual-comp): the CUDA path
against the oracle's dense sum, through mdbf_linear_forward_sum."""
import numpy as np
import pytest
import torch

from oracle import mdbf_oracle as orc
from paper_2512_24545_b200 import inputs, mdbf as M
from helpers import GpuLayer, TOL, TORCH_DT, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2512_24545_b200 import build
    build.build()
    assert torch.cuda.is_available()


def term_specs(d_out, d_in, ks, ls, **kw):
    """Term p: its own seed, inner rank and envelope rank; later terms are smaller (they stand for
    fits to a residual)."""
    base = inputs.qproj(1664)
    return [inputs.scaled(base, name=f"term{p}", d_out=d_out, d_in=d_in, k=k, l=l, seed=70 + p,
                          env_std=0.02 * 0.6 ** p, **kw) for p, (k, l) in enumerate(zip(ks, ls))]


def run_sum(specs, x, act="bf16"):
    T = x.shape[0]
    layers = [GpuLayer(sp, T) for sp in specs]
    try:
        xd = torch.from_numpy(np.ascontiguousarray(x)).to(TORCH_DT[act]).cuda()
        yd = torch.full((T, specs[0].d_out), float("nan"), dtype=TORCH_DT[act], device="cuda")
        acc = torch.full((T, specs[0].d_out), float("nan"), dtype=torch.float32, device="cuda")
        M.mdbf_linear_forward_sum([g.h for g in layers], xd.data_ptr(), yd.data_ptr(), acc.data_ptr(), T,
                                  M.DTYPES[act], torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        for g in layers:
            assert M.mdbf_poll_status(g.h) == 0
        ref = orc.forward_sum([g.oracle_args() for g in layers], x.T.astype(np.float64)).T
        singles = [g.forward(x) for g in layers]
        return yd.to(torch.float32).cpu().numpy(), ref, singles
    finally:
        for g in layers:
            g.close()


@pytest.mark.parametrize("T", [1, 3, 40])
def test_littlebit_format_two_dbf_terms(T):
    specs = term_specs(352, 544, [320, 320], [1, 1])             # (l, P) = (1, 2)
    x = inputs.make_activations(specs[0], T)
    y, ref, _ = run_sum(specs, x)
    assert np.all(np.isfinite(y))
    assert rel_err(y, ref) <= TOL["bf16"]


@pytest.mark.parametrize("T", [1, 5])
def test_three_mdbf_terms_of_different_rank(T):
    specs = term_specs(300, 1000, [257, 128, 64], [16, 4, 2])
    x = inputs.make_activations(specs[0], T)
    y, ref, singles = run_sum(specs, x)
    assert rel_err(y, ref) <= TOL["bf16"]
    # one rounding at the end: at least as close to the oracle as the sum of the separately rounded forwards
    assert rel_err(y, ref) <= rel_err(sum(singles), ref) + 1e-4


@pytest.mark.parametrize("P", [1, 3, 4, 5])
def test_terms_of_one_envelope_rank_at_one_token(P):
    """Up to four terms of one envelope-rank bucket share the first-stage launch and the last term rounds the
    sum into y (store, add, ..., add-and-round); five terms take the term-by-term path with a cast pass."""
    specs = term_specs(300, 1000, [257, 200, 130, 64, 40][:P], [8] * P)
    x = inputs.make_activations(specs[0], 1)
    y, ref, singles = run_sum(specs, x)
    assert np.all(np.isfinite(y))
    assert rel_err(y, ref) <= TOL["bf16"]
    if P == 1:
        np.testing.assert_array_equal(y, singles[0])


def test_fp32_terms_and_single_term():
    t = inputs.tiny()
    specs = [inputs.scaled(t, name="a", seed=1), inputs.scaled(t, name="b", seed=2, env_std=t.env_std * 0.5)]
    x = inputs.make_activations(specs[0], 8)
    y, ref, _ = run_sum(specs, x, act="f32")
    assert rel_err(y, ref) <= TOL["f32"]
    y1, ref1, singles = run_sum(specs[:1], x, act="f32")        # P = 1 is the plain forward
    assert rel_err(y1, ref1) <= TOL["f32"]
    np.testing.assert_array_equal(y1, singles[0])


def test_sum_argument_checks():
    a, b = term_specs(128, 128, [64, 64], [4, 4])
    c = inputs.scaled(a, d_out=256)
    with GpuLayer(a, 1) as ga, GpuLayer(b, 1) as gb, GpuLayer(c, 1) as gc:
        buf = torch.zeros((1, 256), dtype=torch.float32, device="cuda")
        p = buf.data_ptr()
        with pytest.raises(M.MdbfError) as e:
            M.mdbf_linear_forward_sum([ga.h, gc.h], p, p, p, 1, M.BF16)
        assert e.value.status == M.ERR_SHAPE
        with pytest.raises(M.MdbfError) as e:
            M.mdbf_linear_forward_sum([ga.h, ga.h], p, p, p, 1, M.BF16)
        assert e.value.status == M.ERR_INVALID_ARG
        with pytest.raises(M.MdbfError) as e:
            M.mdbf_linear_forward_sum([ga.h, gb.h], p, p, 0, 1, M.BF16)
        assert e.value.status == M.ERR_INVALID_ARG
