"""Every one of the 2^16 sign patterns of a d_out = d_in = 4, k = 2 instance through the library: signs packed by
the library's host packer, one upload, one forward per pattern through the C ABI (fp32 CUDA-core kernels of the
handle-free entry point), compared with the oracle's definition evaluated for all patterns at once; and a stride of
the patterns through mdbf_pack and the one-token tensor-core kernels."""
import itertools

import numpy as np
import pytest
import torch

from oracle import mdbf_oracle as orc
from paper_2512_24545_b200 import inputs, mdbf as M
from helpers import magnitude_bound

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2512_24545_b200 import build
    build.build()
    assert torch.cuda.is_available()


def instance(l, seed=21):
    rng = np.random.default_rng(seed + l)
    d, k = 4, 2
    U_A, V_A = rng.standard_normal((d, l)).astype(np.float32), rng.standard_normal((k, l)).astype(np.float32)
    U_B, V_B = rng.standard_normal((k, l)).astype(np.float32), rng.standard_normal((d, l)).astype(np.float32)
    pats = np.array(list(itertools.product([1, -1], repeat=8)), dtype=np.int8)       # 256 x 8
    return d, k, U_A, V_A, U_B, V_B, pats.reshape(256, d, k), pats.reshape(256, k, d)


@pytest.mark.parametrize("l", [1, 2])
def test_all_sign_patterns_fp32_path(l):
    d, k, U_A, V_A, U_B, V_B, SA_all, SB_all = instance(l)
    T = 3
    x = np.random.default_rng(5).standard_normal((T, d)).astype(np.float32)
    # oracle for all 65 536 patterns: W[a, b] = (S_A[a] (.) U_A V_A^T)(S_B[b] (.) U_B V_B^T)   (Eq. me-dbf-basis)
    UhA = np.stack([orc.modulated_factor(SA_all[a], U_A, V_A) for a in range(256)])  # 256 x d x k
    VhB = np.stack([orc.modulated_factor(SB_all[b], U_B, V_B) for b in range(256)])  # 256 x k x d
    zB = np.einsum("bji,ti->btj", VhB, x.astype(np.float64))                         # 256 x T x k
    y_ref = np.einsum("anj,btj->abtn", UhA, zB)                                      # 256 x 256 x T x d
    # canonical words of every pattern through the host packer, uploaded once
    wA = np.zeros((256 * d, 1), dtype=np.uint32)
    wB = np.zeros((256 * k, 1), dtype=np.uint32)
    M.mdbf_pack_signs(np.ascontiguousarray(SA_all.reshape(256 * d, k)), 256 * d, k, wA, False)
    M.mdbf_pack_signs(np.ascontiguousarray(SB_all.reshape(256 * k, d)), 256 * k, d, wB, False)
    assert np.array_equal(wA.reshape(256, d), np.stack([orc.pack_signs(SA_all[a])[:, 0] for a in range(256)]))
    wAd = torch.from_numpy(wA.view(np.int32)).cuda()
    wBd = torch.from_numpy(wB.view(np.int32)).cuda()
    env = [torch.from_numpy(e).cuda() for e in (U_A, V_A, U_B, V_B)]
    xd = torch.from_numpy(x).cuda()
    yd = torch.full((256, 256, T, d), float("nan"), dtype=torch.float32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    ybase, astride = yd.data_ptr(), 256 * T * d * 4
    for a in range(256):
        pa = wAd.data_ptr() + a * d * 4
        for b in range(256):
            M.mdbf_linear_forward_static(d, d, k, l, M.F32, pa, wBd.data_ptr() + b * k * 4, *[e.data_ptr() for e in env],
                                         xd.data_ptr(), ybase + a * astride + b * T * d * 4, T, M.F32, st)
    torch.cuda.synchronize()
    got = yd.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got))
    num = np.sqrt(((got - y_ref) ** 2).sum(axis=(2, 3)))
    den = np.sqrt((y_ref ** 2).sum(axis=(2, 3)))
    assert np.max(num / np.maximum(den, 1e-30) * (den > 1e-6)) <= 1e-5              # every pattern on its own, fp32 bound
    assert np.max(np.abs(got - y_ref)) <= 1e-5 * np.max(np.abs(y_ref))


@pytest.mark.parametrize("kernel", ["tmem", "i8"])
def test_stride_of_sign_patterns_one_token_tensor_core_kernels(kernel):
    """Every 257th pattern (all 256 values of both factors appear) as a packed layer through the one-token tcgen05
    kernels; with k = 2 nothing averages, so the comparison is the per-element bound."""
    kern = {"tmem": M.KERNEL_TMEM, "i8": M.KERNEL_I8}[kernel]
    roundings = {"tmem": 4, "i8": 1}[kernel]
    for l in (1, 2):
        d, k, U_A, V_A, U_B, V_B, SA_all, SB_all = instance(l)
        spec = inputs.scaled(inputs.qproj(1664), name="bf", d_out=d, d_in=d, k=k, l=l, env_dtype="f16")
        f16 = lambda a: a.astype(np.float16).astype(np.float32)                    # the stored (rounded) envelopes are the layer
        x = np.random.default_rng(6).standard_normal((1, d)).astype(np.float32)
        x = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
        for p in range(0, 65536, 257):
            a, b = p >> 8, p & 255
            lay = {"S_A": SA_all[a], "S_B": SB_all[b], "U_A": f16(U_A), "V_A": f16(V_A), "U_B": f16(U_B), "V_B": f16(V_B)}
            from helpers import GpuLayer
            with GpuLayer(spec, 1, lay=lay) as g:
                y = g.forward(x, kernel=kern)
                ref = g.oracle_forward(x)
                bound = magnitude_bound(g, x)
                assert np.all(np.abs(y - ref) <= (roundings + 1) * 2.0 ** -8 * bound + 1e-30), (l, a, b)
