"""Parity of the one-token integer kernel (packed bits as 8-bit tcgen05 operand, fixed-point scaled input, image +
stage launches) with the CPU oracle: ragged shapes, every envelope-rank bucket it takes, both 16-bit envelope types,
several layers per launch, stages mixed with the bf16 TMEM-operand kernel, repeated calls on one handle."""
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
    return inputs.scaled(inputs.qproj(1664), name="i8", d_out=d_out, d_in=d_in, k=k, l=l, **kw)


@pytest.mark.parametrize("l", [1, 2, 3, 4, 8, 12, 16])
@pytest.mark.parametrize("env", ["f16", "bf16"])
def test_i8_kernel_envelope_ranks(l, env):
    spec = spec_of(419, 1000, 700, l, env_dtype=env)
    x = inputs.make_activations(spec, 1)
    with GpuLayer(spec, 1) as g:
        y = g.forward(x, kernel=M.KERNEL_I8)
        assert M.mdbf_poll_status(g.h) == 0
        assert M.mdbf_last_kernel(g.h) == M.KERNEL_I8 and M.mdbf_last_launch_count(g.h) == 4
        check_parity(g, x, y, roundings=1)                       # fixed-point operands, exact integer sums: only y is rounded
        _, z_ref = orc.forward_staged(*g.oracle_args(), x.T.astype(np.float64))
        assert rel_err(g.intermediate(1), z_ref.T) <= 1e-4       # the intermediate stays fp32
        np.testing.assert_array_equal(y, g.forward(x, kernel=M.KERNEL_I8))       # deterministic, state cleared between calls


@pytest.mark.parametrize("shape", [(1, 1, 1, 1), (31, 127, 33, 2), (129, 1025, 257, 9), (1000, 2100, 1300, 16),
                                   (256, 4096, 512, 16), (2048, 192, 3000, 16), (640, 8192, 100, 16),
                                   (5000, 130, 640, 5)])
def test_i8_kernel_edge_shapes(shape):
    """One row, one column, ragged tails in rows and in the reduction, row-block groups with one to four row blocks,
    reductions split over many CTAs and not at all."""
    d_out, d_in, k, l = shape
    spec = spec_of(d_out, d_in, k, l)
    x = inputs.make_activations(spec, 1)
    with GpuLayer(spec, 1) as g:
        y = g.forward(x, kernel=M.KERNEL_I8)
        assert M.mdbf_poll_status(g.h) == 0
        check_parity(g, x, y, roundings=1)


def test_i8_kernel_outlier_channels_and_zero_input():
    """The fixed-point range follows max |x|: 1 % of the channels 20x larger must not cost the others their
    precision beyond the bound, and an all-zero input gives an all-zero output (scale 0, no division)."""
    spec = spec_of(512, 4096, 768, 16)
    with GpuLayer(spec, 1) as g:
        x = inputs.make_activations(spec, 1)
        check_parity(g, x, g.forward(x, kernel=M.KERNEL_I8), roundings=1)
        x2 = x.copy()
        x2[0, 7] = 3000.0                                        # one huge channel
        check_parity(g, x2, g.forward(x2, kernel=M.KERNEL_I8), roundings=1)
        z = np.zeros_like(x)
        np.testing.assert_array_equal(g.forward(z, kernel=M.KERNEL_I8), np.zeros((1, spec.d_out), dtype=np.float32))
        check_parity(g, x, g.forward(x, kernel=M.KERNEL_I8), roundings=1)        # and the handle is fine afterwards


def test_i8_kernel_matches_the_tmem_kernel():
    spec = spec_of(900, 1536, 1100, 16)
    x = inputs.make_activations(spec, 1)
    with GpuLayer(spec, 1) as g:
        ref = g.oracle_forward(x)
        y8 = g.forward(x, kernel=M.KERNEL_I8)
        yt = g.forward(x, kernel=M.KERNEL_TMEM)
        assert rel_err(y8, ref) <= rel_err(yt, ref)             # one rounding against four
        assert rel_err(y8, yt) <= 2 * TOL["bf16"]


def run_siblings(specs, x, kernel):
    layers = [GpuLayer(sp, 1) for sp in specs]
    try:
        for g in layers:
            M.mdbf_set_kernel(g.h, kernel)
        xd = torch.from_numpy(x).to(torch.bfloat16).cuda()
        ys = [torch.full((1, sp.d_out), float("nan"), dtype=torch.bfloat16, device="cuda") for sp in specs]
        M.mdbf_linear_forward_siblings([g.h for g in layers], xd.data_ptr(), [y.data_ptr() for y in ys], 1, M.BF16,
                                       torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        for g in layers:
            assert M.mdbf_poll_status(g.h) == 0
        assert M.mdbf_last_kernel(layers[0].h) == kernel
        return [(g, y.to(torch.float32).cpu().numpy()) for g, y in zip(layers, ys)]
    except Exception:
        for g in layers:
            g.close()
        raise


@pytest.mark.parametrize("shapes", [[(300, 200), (128, 64)], [(1024, 512), (130, 128), (131, 64), (700, 1100)],
                                    [(640, 640), (2048, 384), (1400, 896), (512, 1152)]])   # row blocks not a multiple of four between full groups
def test_i8_kernel_several_layers_per_launch(shapes):
    """Sibling layers in one set of launches: every CTA walks its share of every layer; layers of different d_out and k."""
    specs = [inputs.scaled(inputs.qproj(1664), name=f"i8s{i}", d_out=do, d_in=640, k=k, l=16, seed=70 + i)
             for i, (do, k) in enumerate(shapes)]
    x = inputs.make_activations(specs[0], 1)
    out = run_siblings(specs, x, M.KERNEL_I8)
    try:
        assert M.mdbf_last_launch_count(out[0][0].h) == 4
        for g, y in out:
            check_parity(g, x, y, roundings=1)
            np.testing.assert_array_equal(y, g.forward(x, kernel=M.KERNEL_I8))   # same digits, same integer sums as alone
    finally:
        for g, _ in out:
            g.close()


@pytest.mark.parametrize("big_stage", ["B", "A"])
def test_stages_mix_kernels(big_stage):
    """AUTO sends a stage with many sign words to the integer kernel and a small one to the TMEM-operand kernel:
    the intermediate passes between them through the handle's fp32 buffer."""
    d_out, d_in = (256, 28672) if big_stage == "B" else (28672, 256)
    spec = spec_of(d_out, d_in, 5376, 16)
    x = inputs.make_activations(spec, 1)
    with GpuLayer(spec, 1) as g:
        y = g.forward(x)
        assert M.mdbf_poll_status(g.h) == 0
        assert M.mdbf_last_launch_count(g.h) == 3               # image + stage launch for the big stage, one for the other
        rows = np.random.default_rng(3).choice(d_out, size=min(d_out, 256), replace=False)
        ref = g.oracle_forward_rows(x, rows)
        assert rel_err(y[:, rows], ref) <= TOL["bf16"]
        y8 = g.forward(x, kernel=M.KERNEL_I8)
        assert rel_err(y8[:, rows], ref) <= TOL["bf16"]
        assert rel_err(y, y8) <= 2 * TOL["bf16"]


def test_group_of_independent_layers():
    """mdbf_linear_forward_group: layers with their own inputs (different d_in) in one set of four launches; each
    output is that layer's forward, bit for bit what the layer gives alone through the same kernel."""
    shapes = [(300, 640, 200), (1024, 384, 512), (130, 2048, 131), (700, 640, 1100), (64, 128, 64)]
    specs = [inputs.scaled(inputs.qproj(1664), name=f"grp{i}", d_out=do, d_in=di, k=k, l=16, seed=90 + i)
             for i, (do, di, k) in enumerate(shapes)]
    layers = [GpuLayer(sp, 1) for sp in specs]
    try:
        xs = [inputs.make_activations(sp, 1) for sp in specs]
        xd = [torch.from_numpy(x).to(torch.bfloat16).cuda() for x in xs]
        ys = [torch.full((1, sp.d_out), float("nan"), dtype=torch.bfloat16, device="cuda") for sp in specs]
        M.mdbf_linear_forward_group([g.h for g in layers], [x.data_ptr() for x in xd], [y.data_ptr() for y in ys], 1, M.BF16,
                                    torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert M.mdbf_last_launch_count(layers[0].h) == 4 and M.mdbf_last_kernel(layers[0].h) == M.KERNEL_I8
        for g, x, y in zip(layers, xs, ys):
            assert M.mdbf_poll_status(g.h) == 0
            got = y.to(torch.float32).cpu().numpy()
            check_parity(g, x, got, roundings=1)
            np.testing.assert_array_equal(got, g.forward(x, kernel=M.KERNEL_I8))
        # three tokens: the same call runs the layers one after the other
        layers3 = [GpuLayer(sp, 3) for sp in specs[:2]]
        try:
            x3 = [inputs.make_activations(sp, 3) for sp in specs[:2]]
            xd3 = [torch.from_numpy(x).to(torch.bfloat16).cuda() for x in x3]
            y3 = [torch.zeros((3, sp.d_out), dtype=torch.bfloat16, device="cuda") for sp in specs[:2]]
            M.mdbf_linear_forward_group([g.h for g in layers3], [x.data_ptr() for x in xd3], [y.data_ptr() for y in y3], 3, M.BF16,
                                        torch.cuda.current_stream().cuda_stream)
            torch.cuda.synchronize()
            for g, x, y in zip(layers3, x3, y3):
                check_parity(g, x, y.to(torch.float32).cpu().numpy())
        finally:
            for g in layers3:
                g.close()
        with pytest.raises(M.MdbfError) as e:
            M.mdbf_linear_forward_group([layers[0].h, layers[0].h], [xd[0].data_ptr()] * 2, [ys[0].data_ptr()] * 2, 1, M.BF16)
        assert e.value.status == M.ERR_INVALID_ARG
    finally:
        for g in layers:
            g.close()
