"""mdbf_linear_forward allocates nothing: free device memory (cudaMemGetInfo) is the same before and after every
variant of the call, including the first call of each kind on a fresh handle; and a handle holds about what its
layer needs (sign words, envelopes, the operand layouts of the default kernels)."""
import numpy as np
import pytest
import torch

from paper_2512_24545_b200 import inputs, mdbf as M
from helpers import GpuLayer, check_parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2512_24545_b200 import build
    build.build()
    assert torch.cuda.is_available()


def free_bytes():
    torch.cuda.synchronize()
    return torch.cuda.mem_get_info()[0]


def test_forward_never_allocates():
    spec = inputs.scaled(inputs.qproj(1664), name="na", d_out=640, d_in=1024, k=512, l=16)
    st = torch.cuda.current_stream().cuda_stream
    with GpuLayer(spec, 300) as g:
        # every buffer of the test exists before the first measurement
        xs = {T: torch.from_numpy(inputs.make_activations(spec, T)).to(torch.bfloat16).cuda() for T in (1, 8, 300)}
        ys = {T: torch.zeros((T, spec.d_out), dtype=torch.bfloat16, device="cuda") for T in (1, 8, 300)}
        buf = torch.zeros(8 * spec.d_in + 8, dtype=torch.bfloat16, device="cuda")
        x_unaligned = buf[1:1 + 8 * spec.d_in].view(8, spec.d_in)
        x_unaligned.copy_(xs[8])
        assert x_unaligned.data_ptr() % 16 == 2
        before = free_bytes()
        calls = [(xs[1], ys[1], 1, M.KERNEL_AUTO), (xs[1], ys[1], 1, M.KERNEL_I8), (xs[1], ys[1], 1, M.KERNEL_TMEM),
                 (xs[8], ys[8], 8, M.KERNEL_AUTO), (x_unaligned, ys[8], 8, M.KERNEL_AUTO), (xs[300], ys[300], 300, M.KERNEL_AUTO),
                 (xs[300], ys[300], 300, M.KERNEL_ALU)]
        for x, y, T, kern in calls:
            M.mdbf_set_kernel(g.h, kern)
            M.mdbf_linear_forward(g.h, x.data_ptr(), y.data_ptr(), T, M.BF16, st)
            assert free_bytes() == before, (T, kern)
        M.mdbf_set_kernel(g.h, M.KERNEL_AUTO)
        assert M.mdbf_poll_status(g.h) == 0
        for T in (1, 8, 300):                                    # and the results are the layer's
            x = xs[T].to(torch.float32).cpu().numpy()
            M.mdbf_linear_forward(g.h, xs[T].data_ptr(), ys[T].data_ptr(), T, M.BF16, st)
            torch.cuda.synchronize()
            check_parity(g, x, ys[T].to(torch.float32).cpu().numpy())
    # a forced expanded order without its scratch is an error, not an allocation; mdbf_set_kernel(PREFILL) is the one
    # place that allocates that scratch
    with GpuLayer(spec, 300) as g2:
        g2.h_kernel = None
        before = free_bytes()
        M.mdbf_set_kernel(g2.h, M.KERNEL_PREFILL)
        assert free_bytes() < before
        mid = free_bytes()
        M.mdbf_linear_forward(g2.h, xs[8].data_ptr(), ys[8].data_ptr(), 8, M.BF16, st)
        assert free_bytes() == mid


def test_handle_footprint_is_about_one_bit_per_sign():
    """4096 x 4096, k = 1664, l = 16, one token: the handle may hold its signs once (plus the operand layouts of the
    envelopes and the scratch of the one-token kernels), not several copies of them."""
    spec = inputs.qproj(1664)
    lay = inputs.make_layer(spec)
    args = [torch.from_numpy(np.ascontiguousarray(lay[n])).cuda() for n in ("S_A", "S_B", "U_A", "V_A", "U_B", "V_B")]
    torch.cuda.synchronize()
    before = free_bytes()
    h = M.mdbf_pack(spec.d_out, spec.d_in, spec.k, spec.l, M.DTYPES[spec.env_dtype], 1, *[a.data_ptr() for a in args],
                    inputs_on_device=True)
    used = before - free_bytes()
    M.mdbf_destroy(h)
    signs = spec.k * (spec.d_in + spec.d_out) // 8
    envelopes = 2 * spec.l * (spec.d_in + spec.d_out + 2 * spec.k)
    # bf16 V tile images of the TMEM-operand kernel, operand images + 64-bit accumulators of the integer kernel, fp32 z
    layouts = 2 * 16 * (spec.d_in + spec.k) + 48 * (spec.d_in + spec.k) + 8 * (spec.k + spec.d_out) + 4 * spec.k
    need = signs + envelopes + layouts
    assert used <= 1.10 * need + (4 << 20), (used, need)         # cudaMalloc rounds small buffers up: 4 MiB of slack
