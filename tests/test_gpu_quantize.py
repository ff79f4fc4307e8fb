"""The layer-wise pipeline end to end on the GPU (truncated SVD, MSVID initialisation, ADMM refinement, pack, forward)
against the same pipeline assembled from the oracle's functions."""
import numpy as np
import pytest
import torch

from oracle import mdbf_oracle as orc
from paper_2512_24545_b200 import mdbf as M, quantize

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2512_24545_b200 import build
    build.build()
    assert torch.cuda.is_available()


def oracle_pipeline(W, R, l, n_alternations, n_inner, rho_scale):
    Uu, s, Vt = np.linalg.svd(W, full_matrices=False)
    U0, V0 = Uu[:, :R] * np.sqrt(s[:R]), Vt[:R].T * np.sqrt(s[:R])
    SU, A, B = orc.msvid(U0, l)
    SV, C, D = orc.msvid(V0, l)
    U, V = SU * (A @ B.T), SV * (C @ D.T)
    init = np.linalg.norm(W - U @ V.T) / np.linalg.norm(W)
    LU, LV = np.zeros_like(U), np.zeros_like(V)
    for _ in range(n_alternations):
        U, LU, _, _ = orc.admm_factor_update(W, V, U, LU, rho_scale * np.sum(V ** 2) / R, l, n_inner)
        V, LV, _, _ = orc.admm_factor_update(W.T, U, V, LV, rho_scale * np.sum(U ** 2) / R, l, n_inner)
    return init, np.linalg.norm(W - U @ V.T) / np.linalg.norm(W)


def test_quantize_pack_forward():
    rng = np.random.default_rng(70)
    N, Mc, R, l = 384, 320, 128, 8
    W = (rng.standard_normal((N, 40)) @ rng.standard_normal((40, Mc)) / 6 + 0.3 * rng.standard_normal((N, Mc))).astype(np.float32)
    q = quantize.quantize_layer(torch.from_numpy(W).cuda(), R, l, n_alternations=2, n_inner=3, n_iter=10, rho_scale=3.0)
    init_o, final_o = oracle_pipeline(W.astype(np.float64), R, l, 2, 3, 3.0)
    assert q.err_svd < q.err_init
    assert abs(q.err_init - init_o) <= 0.03 * init_o            # the initialisation is the oracle's (exact SVDs there)
    assert final_o < init_o                                     # the refinement refines
    assert q.err_final <= q.err_init and abs(q.err_final - final_o) <= 0.05 * final_o
    # the compact factors are the dense ones the refinement ended with
    Wq = q.dense().cpu().numpy()
    assert abs(np.linalg.norm(W - Wq) / np.linalg.norm(W) - q.err_final) <= 1e-4
    # every factor has the format: +-1 masks, rank-l envelopes
    assert set(np.unique(q.S_A.cpu().numpy())) <= {-1, 1} and set(np.unique(q.S_B.cpu().numpy())) <= {-1, 1}
    assert q.S_A.shape == (N, R) and q.S_B.shape == (R, Mc)
    # and as a layer of the library it reconstructs and multiplies like the oracle says (fp32 envelopes: no storage rounding)
    h = q.pack(env_dtype=M.F32, max_T=8)
    try:
        Wd = torch.empty((N, Mc), dtype=torch.float32, device="cuda")
        M.mdbf_reconstruct(h, Wd.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        ref = orc.reconstruct(*[t.cpu().numpy() for t in (q.S_A, q.S_B, q.U_A, q.V_A, q.U_B, q.V_B)])
        assert orc.rel_frobenius(Wd.cpu().numpy(), ref) <= 1e-6
        x = rng.standard_normal((5, Mc)).astype(np.float32)
        xd = torch.from_numpy(x).cuda()
        yd = torch.empty((5, N), dtype=torch.float32, device="cuda")
        M.mdbf_linear_forward(h, xd.data_ptr(), yd.data_ptr(), 5, M.F32, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert orc.rel_frobenius(yd.cpu().numpy(), (ref @ x.T.astype(np.float64)).T) <= 1e-5
        # the quantized layer approximates the original one as well as its weights do
        y_true = (W.astype(np.float64) @ x.T.astype(np.float64)).T
        assert orc.rel_frobenius(yd.cpu().numpy(), y_true) <= 1.5 * q.err_final
    finally:
        M.mdbf_destroy(h)


def test_initialisation_only_and_argument_checks():
    rng = np.random.default_rng(71)
    W = rng.standard_normal((200, 260)).astype(np.float32)
    q = quantize.quantize_layer(torch.from_numpy(W).cuda(), 64, 4, n_alternations=0)
    assert q.err_final == q.err_init and np.isfinite(q.err_init)
    with pytest.raises(ValueError):
        quantize.quantize_layer(torch.from_numpy(W).cuda(), 300, 4)
    with pytest.raises(ValueError):
        quantize.quantize_layer(torch.from_numpy(W), 64, 4)
