"""Sibling projections on a shared input (q/k/v, gate/up): the fused one-token launches and the
sequential fallback against the oracle and against separate forwards."""
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


def sib_specs(d_in, shapes, l=16, **kw):
    base = inputs.qproj(1664)
    return [inputs.scaled(base, name=f"sib{i}", d_out=do, d_in=d_in, k=k, l=l, seed=90 + i, **kw)
            for i, (do, k) in enumerate(shapes)]


def run_siblings(specs, x):
    T = x.shape[0]
    layers = [GpuLayer(sp, max(T, 1)) for sp in specs]
    try:
        xd = torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16).cuda()
        ys = [torch.full((T, sp.d_out), float("nan"), dtype=torch.bfloat16, device="cuda") for sp in specs]
        M.mdbf_linear_forward_siblings([g.h for g in layers], xd.data_ptr(), [y.data_ptr() for y in ys], T, M.BF16,
                                       torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        out = []
        for g, y in zip(layers, ys):
            assert M.mdbf_poll_status(g.h) == 0
            got = y.to(torch.float32).cpu().numpy()
            out.append((got, g.oracle_forward(x), g.forward(x)))
        return out
    finally:
        for g in layers:
            g.close()


@pytest.mark.parametrize("shapes", [[(384, 320), (96, 64), (96, 64)],              # q, k, v like: one big, two small
                                    [(700, 257), (700, 257)],                        # gate, up like
                                    [(130, 100), (64, 33), (257, 129), (31, 31), (300, 65)]])   # five: two groups
def test_fused_siblings_one_token(shapes):
    specs = sib_specs(544, shapes)
    x = inputs.make_activations(specs[0], 1)
    for got, ref, single in run_siblings(specs, x):
        assert np.all(np.isfinite(got))
        assert rel_err(got, ref) <= TOL["bf16"]
        assert rel_err(got, single) <= 1e-3                   # same arithmetic up to the order of the cluster reduction


@pytest.mark.parametrize("shapes", [[(9600, 2048), (9600, 2048)],       # 150 row blocks on 148 SMs: two go to the short launch
                                    [(19300, 2100)]])                    # one layer, 151 row blocks, ragged last block
def test_last_partial_wave_goes_to_a_second_launch(shapes):
    """Stage A has a few more row blocks than SMs: the row blocks of the last, nearly empty wave run in a
    second launch with the reduction split over a cluster.  Every output row must still be written once."""
    specs = sib_specs(256, shapes)
    x = inputs.make_activations(specs[0], 1)
    for (got, ref, single), sp in zip(run_siblings(specs, x), specs):
        assert np.all(np.isfinite(got))
        assert rel_err(got, ref) <= TOL["bf16"]
        assert rel_err(got[:, -400:], ref[:, -400:]) <= TOL["bf16"]      # the rows the second launch wrote
        assert rel_err(got, single) <= 1e-3


def test_second_launch_is_counted():
    spec = sib_specs(256, [(19300, 2100)])[0]
    x = inputs.make_activations(spec, 1)
    with GpuLayer(spec, 1) as g:
        g.forward(x)
        assert M.mdbf_last_launch_count(g.h) == 3             # stage B, stage A main part, stage A last row blocks


def test_siblings_fall_back_to_separate_forwards():
    specs = sib_specs(256, [(128, 128), (64, 96)])
    x = inputs.make_activations(specs[0], 3)                  # three tokens: not fused
    for got, ref, single in run_siblings(specs, x):
        assert rel_err(got, ref) <= TOL["bf16"]
        np.testing.assert_array_equal(got, single)
    mixed = sib_specs(256, [(128, 128)], l=16) + sib_specs(256, [(64, 96)], l=4)     # different envelope-rank buckets
    x1 = inputs.make_activations(mixed[0], 1)
    for got, ref, single in run_siblings(mixed, x1):
        assert rel_err(got, ref) <= TOL["bf16"]


def test_siblings_argument_checks():
    a, b = sib_specs(256, [(128, 128), (64, 96)])
    c = inputs.scaled(a, d_in=128)
    with GpuLayer(a, 1) as ga, GpuLayer(b, 1) as gb, GpuLayer(c, 1) as gc:
        buf = torch.zeros((1, 256), dtype=torch.bfloat16, device="cuda")
        p = buf.data_ptr()
        with pytest.raises(M.MdbfError) as e:
            M.mdbf_linear_forward_siblings([ga.h, gc.h], p, [p, p], 1, M.BF16)
        assert e.value.status == M.ERR_SHAPE
        with pytest.raises(M.MdbfError) as e:
            M.mdbf_linear_forward_siblings([ga.h, ga.h], p, [p, p], 1, M.BF16)
        assert e.value.status == M.ERR_INVALID_ARG
        with pytest.raises(M.MdbfError) as e:
            M.mdbf_linear_forward_siblings([ga.h, gb.h], p, [p, 0], 1, M.BF16)
        assert e.value.status == M.ERR_INVALID_ARG
        with pytest.raises(M.MdbfError) as e:
            M.mdbf_linear_forward_siblings([ga.h, gb.h], p, [p, p], 2, M.BF16)     # max_T = 1
        assert e.value.status == M.ERR_SHAPE
