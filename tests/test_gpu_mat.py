"""Parity of the materialised-envelope kernel (W_hat tiles rebuilt on the fly from Eq. me-dbf-basis,
one GEMM of width T) with the CPU oracle: shapes that span several 128-row tiles, several K
blocks, several token tiles and ragged tails in every dimension."""
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
    return inputs.scaled(inputs.qproj(1664), name="mat", d_out=d_out, d_in=d_in, k=k, l=l, outliers=False, **kw)


@pytest.mark.parametrize("l,T", [(16, 16), (16, 48), (16, 5), (16, 2), (4, 64), (4, 100), (1, 256), (1, 300),
                                 (3, 40), (8, 33), (20, 9), (32, 11), (16, 600), (32, 130), (20, 300), (2, 65)])
def test_mat_kernel_small_shapes(l, T):
    spec = spec_of(384, 576, 256, l)
    x = inputs.make_activations(spec, T)
    with GpuLayer(spec, T) as g:
        ref = g.oracle_forward(x)
        y = g.forward(x, kernel=M.KERNEL_MAT)
        assert M.mdbf_poll_status(g.h) == 0
        check_parity(g, x, y, ref)                               # whole array, every 128-row block, every element
        _, z_ref = orc.forward_staged(*g.oracle_args(), x.T.astype(np.float64))
        assert rel_err(g.intermediate(T), z_ref.T) <= TOL["bf16"]


@pytest.mark.parametrize("shape", [(1, 8, 1, 1), (100, 72, 50, 2), (129, 72, 130, 16), (300, 1000, 260, 5),
                                   (130, 64, 65, 17)])
def test_mat_kernel_ragged_shapes(shape):
    d_out, d_in, k, l = shape
    spec = spec_of(d_out, d_in, k, l)
    x = inputs.make_activations(spec, 19)
    with GpuLayer(spec, 19) as g:
        y = g.forward(x, kernel=M.KERNEL_MAT)
        assert M.mdbf_poll_status(g.h) == 0
        # a layer with a few terms per output cannot average its four bf16 roundings (W_hat of either stage, z, y):
        # there the per-element bound is the assertion
        check_parity(g, x, y, averaging=k >= 8)


@pytest.mark.parametrize("shape", [(128, 2048, 1024, 8, 8), (256, 1100 * 8, 520, 16, 40), (200, 4096, 136, 3, 2)])
def test_mat_kernel_split_reduction(shape):
    """Few tokens and few row blocks: the reduction is split over a cluster and summed through shared memory."""
    d_out, d_in, k, l, T = shape
    spec = spec_of(d_out, d_in, k, l)
    x = inputs.make_activations(spec, T)
    with GpuLayer(spec, T) as g:
        y = g.forward(x, kernel=M.KERNEL_MAT)
        assert M.mdbf_poll_status(g.h) == 0
        check_parity(g, x, y)
        np.testing.assert_array_equal(y, g.forward(x, kernel=M.KERNEL_MAT))     # deterministic summation order


@pytest.mark.parametrize("env_dtype,T", [("f16", 64), ("bf16", 64), ("f16", 200), ("bf16", 200)])
def test_mat_kernel_envelope_types_and_other_kernels(env_dtype, T):
    spec = spec_of(256, 512, 256, 16, env_dtype=env_dtype)
    x = inputs.make_activations(spec, T)
    with GpuLayer(spec, T) as g:
        ref = g.oracle_forward(x)
        y_mat = g.forward(x, kernel=M.KERNEL_MAT)
        y_pf = g.forward(x, kernel=M.KERNEL_PREFILL)
        assert rel_err(y_mat, ref) <= TOL["bf16"] and rel_err(y_pf, ref) <= TOL["bf16"]
        assert rel_err(y_mat, y_pf) <= 2 * TOL["bf16"]
        # repeated calls give the same bits
        np.testing.assert_array_equal(y_mat, g.forward(x, kernel=M.KERNEL_MAT))


def test_mat_kernel_rejects_what_it_cannot_take():
    spec = spec_of(128, 100, 64, 4)                       # d_in not a multiple of 8: no tensor map over x
    x = inputs.make_activations(spec, 8)
    with GpuLayer(spec, 8) as g:
        with pytest.raises(M.MdbfError) as e:
            g.forward(x, kernel=M.KERNEL_MAT)
        assert e.value.status == M.ERR_SHAPE
        assert rel_err(g.forward(x), g.oracle_forward(x)) <= TOL["bf16"]       # AUTO still serves it
    spec = spec_of(128, 128, 64, 4)
    x1 = inputs.make_activations(spec, 1)
    with GpuLayer(spec, 8) as g:
        with pytest.raises(M.MdbfError) as e:
            g.forward(x1, kernel=M.KERNEL_MAT)                                  # one token
        assert e.value.status == M.ERR_SHAPE


def test_auto_dispatch_reports_its_kernel_and_serves_unaligned_x():
    spec = spec_of(256, 512, 256, 16)
    with GpuLayer(spec, 64) as g:
        assert M.mdbf_last_kernel(g.h) == 0
        x1 = inputs.make_activations(spec, 1)
        g.forward(x1)
        assert M.mdbf_last_kernel(g.h) == M.KERNEL_TMEM
        x8 = inputs.make_activations(spec, 8)
        y8 = g.forward(x8)
        assert M.mdbf_last_kernel(g.h) == M.KERNEL_MAT
        ref = g.oracle_forward(x8)
        assert rel_err(y8, ref) <= TOL["bf16"]
        # x two bytes off a 16-byte boundary: no tensor map over it and no scratch for the expanded order on this
        # handle: the CUDA-core kernel serves the call (a forward never allocates); after mdbf_set_kernel(PREFILL)
        # has built that scratch, the library's own choice for such an x is the expanded order
        buf = torch.zeros(8 * spec.d_in + 8, dtype=torch.bfloat16, device="cuda")
        xd = buf[1:1 + 8 * spec.d_in].view(8, spec.d_in)
        xd.copy_(torch.from_numpy(x8).to(torch.bfloat16))
        assert xd.data_ptr() % 16 == 2
        yd = torch.zeros((8, spec.d_out), dtype=torch.bfloat16, device="cuda")
        M.mdbf_linear_forward(g.h, xd.data_ptr(), yd.data_ptr(), 8, M.BF16, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert M.mdbf_last_kernel(g.h) == M.KERNEL_ALU
        assert rel_err(yd.to(torch.float32).cpu().numpy(), ref) <= TOL["bf16"]
        M.mdbf_set_kernel(g.h, M.KERNEL_PREFILL)
        M.mdbf_set_kernel(g.h, M.KERNEL_AUTO)
        yd.zero_()
        M.mdbf_linear_forward(g.h, xd.data_ptr(), yd.data_ptr(), 8, M.BF16, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert M.mdbf_last_kernel(g.h) == M.KERNEL_PREFILL
        assert rel_err(yd.to(torch.float32).cpu().numpy(), ref) <= TOL["bf16"]
    with GpuLayer(inputs.tiny(), 8) as g:                                      # fp32 layer
        g.forward(inputs.make_activations(inputs.tiny(), 8))
        assert M.mdbf_last_kernel(g.h) == M.KERNEL_ALU


def _random_shapes(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        d_out = int(rng.integers(1, 700))
        d_in = 8 * int(rng.integers(1, 90))                      # the tensor map over x needs a multiple of 8
        k = int(rng.integers(1, 500))
        l = int(rng.choice([1, 2, 3, 5, 8, 13, 16, 17, 24, 32]))
        T = int(rng.choice([2, 3, 7, 16, 17, 31, 48, 64, 65, 100, 255, 256, 257, 400]))
        out.append((d_out, d_in, k, l, T))
    return out


@pytest.mark.parametrize("shape", _random_shapes(24, seed=2512))
def test_mat_kernels_seeded_random_shapes(shape):
    """Ragged sizes in every dimension at once, through AUTO (small-tile kernel up to 64 tokens, large-tile above)."""
    d_out, d_in, k, l, T = shape
    spec = spec_of(d_out, d_in, k, l)
    x = inputs.make_activations(spec, T)
    with GpuLayer(spec, T) as g:
        y = g.forward(x)
        assert M.mdbf_last_kernel(g.h) == M.KERNEL_MAT
        assert M.mdbf_poll_status(g.h) == 0
        assert np.all(np.isfinite(y))
        check_parity(g, x, y, averaging=k >= 32)                # few terms per output: the per-element bound alone
