"""Multi-Envelope SVID on the GPU (mdbf_msvid, Eq. msvid-def) against the oracle: the sign mask bit for bit, and the
truncated envelope through what is unique about it - the singular values and the error of Theorem 1
(Eq. rankl-error), which the exact TSVD attains and no rank-l envelope can beat.  The factors themselves are not
compared: they are unique only up to signs and to rotations among equal singular values, and the GPU computes
them by subspace iteration, not by a full SVD."""
import numpy as np
import pytest
import torch

from oracle import mdbf_oracle as orc
from paper_2512_24545_b200 import inputs, mdbf as M

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2512_24545_b200 import build
    build.build()
    assert torch.cuda.is_available()


def run_msvid(Z, l, n_iter, Q0=None, seed=11):
    rows, cols = Z.shape
    Q0 = inputs.make_start_block(cols, l, seed) if Q0 is None else Q0
    Zd = torch.from_numpy(np.ascontiguousarray(Z, dtype=np.float32)).cuda()
    Qd = torch.from_numpy(np.ascontiguousarray(Q0, dtype=np.float32)).cuda()
    nwords = (cols + 31) // 32
    Sd = torch.full((rows, nwords), -1, dtype=torch.int32, device="cuda")
    Ud = torch.full((rows, l), float("nan"), dtype=torch.float32, device="cuda")
    Vd = torch.full((cols, l), float("nan"), dtype=torch.float32, device="cuda")
    sd = torch.full((l,), float("nan"), dtype=torch.float32, device="cuda")
    nbytes = M.mdbf_msvid_workspace_bytes(rows, cols, l)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    M.mdbf_msvid(Zd.data_ptr(), rows, cols, l, n_iter, Qd.data_ptr(), Sd.data_ptr(), Ud.data_ptr(), Vd.data_ptr(), sd.data_ptr(),
                 ws.data_ptr(), nbytes, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return (Sd.cpu().numpy().view(np.uint32), Ud.cpu().numpy().astype(np.float64), Vd.cpu().numpy().astype(np.float64),
            sd.cpu().numpy().astype(np.float64))


def envelope_error(Z, U, V):
    return np.linalg.norm(np.abs(Z.astype(np.float64)) - U @ V.T)


# shapes whose column count is a multiple of four run the tensor-core products (ragged last row block and K block
# included), the others the scalar kernels; l = 8 and 32 take the remaining operand widths
@pytest.mark.parametrize("shape,l", [(s, l) for s in [(300, 517), (1024, 768), (129, 33), (64, 2000), (2000, 64), (33, 40)]
                                     for l in (1, 4, 16)] + [((333, 516), 8), ((333, 516), 32), ((1000, 260), 8), ((1000, 260), 32),
                                                             ((515, 1028), 16)])
def test_sign_mask_exact_and_envelope_near_the_optimum(shape, l):
    rows, cols = shape
    Z = inputs.make_factor_matrix(rows, cols, seed=5)
    S_ref, _, _ = orc.msvid(Z, l)
    sv = np.linalg.svd(np.abs(Z.astype(np.float64)), compute_uv=False)
    tail = np.sqrt(np.sum(sv[l:] ** 2))                                    # Eq. rankl-error
    Sp, U, V, s = run_msvid(Z, l, n_iter=8)
    # the mask: integer work, bit for bit (sign(0) = sign(-0) = +1, the tiny negative entry is -1)
    np.testing.assert_array_equal(Sp, orc.pack_signs(S_ref))
    # singular values: the leading one has converged; every estimate is a lower bound of the exact value (Ritz
    # values of a projection) and not far below it after eight iterations
    assert np.all(np.isfinite(U)) and np.all(np.isfinite(V)) and np.all(np.isfinite(s))
    assert abs(s[0] - sv[0]) <= 2e-5 * sv[0]
    assert np.all(s <= sv[:l] * (1 + 2e-5))
    assert np.all(s >= 0.80 * sv[:l])
    assert np.all(np.diff(s) <= 1e-6 * sv[0])                              # descending
    # the envelope: no rank-l matrix beats the tail of Theorem 1, and the iteration ends within 1 % of it
    err = envelope_error(Z, U, V)
    assert err >= tail * (1 - 1e-5)
    assert err <= tail * 1.01 + 1e-5 * sv[0]
    # remodulated with the mask the error is the same number (Eq. envelope-isometry)
    S = orc.unpack_signs(Sp, cols).astype(np.float64)
    assert abs(np.linalg.norm(Z.astype(np.float64) - S * (U @ V.T)) - err) <= 1e-9 * sv[0]
    # balanced factors: both columns of a pair carry the square root of their singular value
    np.testing.assert_allclose(np.linalg.norm(U, axis=0), np.sqrt(s), rtol=2e-4)
    np.testing.assert_allclose(np.linalg.norm(V, axis=0), np.sqrt(s), rtol=2e-4)


def test_bench_size_factor_properties():
    """The factor bench.py times (28672 x 6016, l = 16, four iterations), too large for a full SVD in the test: the mask of
    sampled rows bit for bit, and what holds for the result at any size - singular values in descending order, balanced
    column norms, and the residual of every sampled row orthogonal to the right factors (U is the product of |Z| with an
    orthonormal basis of V's range, so (|z_i| - u_i V^T) V = 0 up to rounding), which pins the last pass over Z."""
    rows, cols, l = 28672, 6016, 16
    Z = inputs.make_factor_matrix(rows, cols, seed=8)
    Sp, U, V, s = run_msvid(Z, l, n_iter=4, seed=8)
    pick = np.random.default_rng(3).choice(rows, size=64, replace=False)
    np.testing.assert_array_equal(Sp[pick], orc.pack_signs(np.where(Z[pick] >= 0, 1, -1).astype(np.int8)))
    assert np.all(np.isfinite(s)) and np.all(np.diff(s) <= 1e-6 * s[0]) and s[-1] > 0
    np.testing.assert_allclose(np.linalg.norm(U, axis=0), np.sqrt(s), rtol=5e-4)
    np.testing.assert_allclose(np.linalg.norm(V, axis=0), np.sqrt(s), rtol=5e-4)
    E = np.abs(Z[pick].astype(np.float64))
    resid = E - U[pick] @ V.T
    assert np.max(np.abs(resid @ V)) <= 2e-4 * np.max(np.abs(E @ V))
    # the leading singular value against a few steps of the power method in fp64 on a block of rows is a lower bound check:
    # sigma_1 of the whole matrix is at least that of any block of its rows
    blk = np.abs(Z[:2048].astype(np.float64))
    v = np.ones(cols) / np.sqrt(cols)
    for _ in range(6):
        v = blk.T @ (blk @ v)
        v /= np.linalg.norm(v)
    assert s[0] >= np.linalg.norm(blk @ v) * (1 - 1e-6)


def test_tensor_core_and_scalar_products_agree():
    """The same matrix at a 16-byte aligned address (tensor-core products, three-term TF32 split) and four bytes further on
    (the scalar fp32 kernels): the same mask, and singular values that agree to fp32 accuracy."""
    rows, cols, l = 700, 1028, 16
    Z = inputs.make_factor_matrix(rows, cols, seed=6)
    Q0 = inputs.make_start_block(cols, l, 12)
    buf = torch.zeros(rows * cols + 1, dtype=torch.float32, device="cuda")
    Zt = torch.from_numpy(Z).cuda().reshape(-1)
    nwords = (cols + 31) // 32
    nbytes = M.mdbf_msvid_workspace_bytes(rows, cols, l)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    Qd = torch.from_numpy(Q0).cuda()
    res = []
    for off in (0, 1):
        buf.zero_()
        buf[off:off + rows * cols] = Zt
        Sd = torch.zeros((rows, nwords), dtype=torch.int32, device="cuda")
        Ud = torch.zeros((rows, l), dtype=torch.float32, device="cuda")
        Vd = torch.zeros((cols, l), dtype=torch.float32, device="cuda")
        sd = torch.zeros((l,), dtype=torch.float32, device="cuda")
        assert (buf.data_ptr() + 4 * off) % 16 == (0 if off == 0 else 4)
        M.mdbf_msvid(buf.data_ptr() + 4 * off, rows, cols, l, 6, Qd.data_ptr(), Sd.data_ptr(), Ud.data_ptr(), Vd.data_ptr(),
                     sd.data_ptr(), ws.data_ptr(), nbytes, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        res.append((Sd.cpu().numpy(), sd.cpu().numpy().astype(np.float64), Ud.cpu().numpy().astype(np.float64),
                    Vd.cpu().numpy().astype(np.float64)))
    np.testing.assert_array_equal(res[0][0], res[1][0])
    np.testing.assert_allclose(res[0][1], res[1][1], rtol=2e-5)
    e0, e1 = envelope_error(Z, res[0][2], res[0][3]), envelope_error(Z, res[1][2], res[1][3])
    assert abs(e0 - e1) <= 1e-5 * e1


@pytest.mark.parametrize("trial", range(12))
def test_random_shapes_both_product_paths(trial):
    """Randomly drawn sizes with a column count that the tensor-core path accepts, each run twice: at an aligned address
    (tensor-core products) and four bytes further on (scalar fp32 kernels).  Same mask, singular values and envelope error
    that agree to the accuracy of the split (a few 1e-6 of the norm); every third case under a given mask."""
    rng = np.random.default_rng(1200 + trial)
    rows, cols = int(rng.integers(1, 1200)), 4 * int(rng.integers(1, 400))
    l = int(min(rng.choice([1, 2, 3, 4, 7, 8, 13, 16, 20, 32]), rows, cols))
    masked = trial % 3 == 2
    Z = inputs.make_factor_matrix(rows, cols, seed=1000 + trial)
    S = inputs.make_signs(rows, cols, seed=trial, stream="S_A") if masked else None
    Qd = torch.from_numpy(inputs.make_start_block(cols, l, 2000 + trial)).cuda()
    buf = torch.zeros(rows * cols + 1, dtype=torch.float32, device="cuda")
    Zt = torch.from_numpy(Z).cuda().reshape(-1)
    nwords = (cols + 31) // 32
    nbytes = M.mdbf_msvid_workspace_bytes(rows, cols, l)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    res = []
    for off in (0, 1):
        buf.zero_()
        buf[off:off + rows * cols] = Zt
        Sd = (torch.from_numpy(orc.pack_signs(S).view(np.int32)).cuda() if masked
              else torch.zeros((rows, nwords), dtype=torch.int32, device="cuda"))
        Ud = torch.zeros((rows, l), dtype=torch.float32, device="cuda")
        Vd = torch.zeros((cols, l), dtype=torch.float32, device="cuda")
        sd = torch.zeros((l,), dtype=torch.float32, device="cuda")
        if masked:
            M.mdbf_project_fixed_mask(buf.data_ptr() + 4 * off, Sd.data_ptr(), rows, cols, l, 5, Qd.data_ptr(), Ud.data_ptr(), Vd.data_ptr(),
                                      sd.data_ptr(), ws.data_ptr(), nbytes, st)
        else:
            M.mdbf_msvid(buf.data_ptr() + 4 * off, rows, cols, l, 5, Qd.data_ptr(), Sd.data_ptr(), Ud.data_ptr(), Vd.data_ptr(), sd.data_ptr(),
                         ws.data_ptr(), nbytes, st)
        torch.cuda.synchronize()
        res.append((Sd.cpu().numpy(), sd.cpu().numpy().astype(np.float64), Ud.cpu().numpy().astype(np.float64),
                    Vd.cpu().numpy().astype(np.float64)))
    np.testing.assert_array_equal(res[0][0], res[1][0])
    assert np.all(np.isfinite(res[0][1]))
    np.testing.assert_allclose(res[0][1], res[1][1], rtol=5e-4, atol=1e-6 * res[1][1][0])
    E = Z.astype(np.float64) * S if masked else np.abs(Z.astype(np.float64))
    e0, e1 = np.linalg.norm(E - res[0][2] @ res[0][3].T), np.linalg.norm(E - res[1][2] @ res[1][3].T)
    assert abs(e0 - e1) <= 2e-4 * e1 + 1e-5 * np.linalg.norm(E)


def test_error_decreases_with_envelope_rank_and_with_iterations():
    Z = inputs.make_factor_matrix(700, 900, seed=6)
    errs_l = [envelope_error(Z, *run_msvid(Z, l, n_iter=6)[1:3]) for l in (1, 2, 4, 8, 16, 32)]
    assert all(b <= a * (1 + 1e-6) for a, b in zip(errs_l, errs_l[1:]))   # F_1(S) is inside F_l(S): Theorem 1's remark
    errs_it = [envelope_error(Z, *run_msvid(Z, 16, n_iter=n)[1:3]) for n in (1, 2, 4, 8, 16)]
    assert all(b <= a * (1 + 1e-6) for a, b in zip(errs_it, errs_it[1:]))
    sv = np.linalg.svd(np.abs(Z.astype(np.float64)), compute_uv=False)
    assert errs_it[-1] <= np.sqrt(np.sum(sv[16:] ** 2)) * 1.005


def test_envelope_of_exact_low_rank_is_reproduced():
    """|Z| of rank 3 and l = 4: the block is wider than the rank, the fourth singular value is zero, the first three
    reproduce |Z| (and Z, with the mask) to fp32 accuracy."""
    rng = np.random.default_rng(17)
    E = np.abs(rng.standard_normal((257, 3))) @ np.abs(rng.standard_normal((3, 190)))
    S = np.where(rng.random((257, 190)) < 0.5, -1.0, 1.0)
    Z = (S * E).astype(np.float32)
    Sp, U, V, s = run_msvid(Z, 4, n_iter=3)
    np.testing.assert_array_equal(Sp, orc.pack_signs(np.where(Z >= 0, 1, -1).astype(np.int8)))
    sv = np.linalg.svd(np.abs(Z.astype(np.float64)), compute_uv=False)
    np.testing.assert_allclose(s[:3], sv[:3], rtol=2e-5)
    assert s[3] <= 1e-3 * sv[0]
    assert envelope_error(Z, U, V) <= 2e-5 * np.linalg.norm(Z)
    Sm = orc.unpack_signs(Sp, 190).astype(np.float64)
    assert np.linalg.norm(Z - Sm * (U @ V.T)) <= 2e-5 * np.linalg.norm(Z)


def test_full_size_factor():
    """4096 x 4096, l = 16: the mask against the oracle on every row, the singular values against the full SVD, the
    envelope error through ||A - A Q Q^T||^2 = ||A||^2 - sum s_t^2 (Q orthonormal) against Theorem 1's tail."""
    Z = inputs.make_factor_matrix(4096, 4096, seed=7)
    Sp, U, V, s = run_msvid(Z, 16, n_iter=4)
    np.testing.assert_array_equal(Sp, orc.pack_signs(np.where(Z >= 0, 1, -1).astype(np.int8)))
    A = np.abs(Z.astype(np.float64))
    sv = np.linalg.svd(A, compute_uv=False)
    assert abs(s[0] - sv[0]) <= 2e-5 * sv[0]
    assert np.all(s <= sv[:16] * (1 + 2e-5)) and np.all(s >= 0.8 * sv[:16])
    tail2 = np.sum(sv[16:] ** 2)
    err2 = np.sum(A * A) - np.sum(s ** 2)
    assert tail2 * (1 - 1e-4) <= err2 <= tail2 * 1.01


def run_projection(Z, S, l, n_iter, seed=11):
    rows, cols = Z.shape
    Zd = torch.from_numpy(np.ascontiguousarray(Z, dtype=np.float32)).cuda()
    Qd = torch.from_numpy(inputs.make_start_block(cols, l, seed)).cuda()
    Sd = torch.from_numpy(orc.pack_signs(S).view(np.int32)).cuda()
    Ud = torch.full((rows, l), float("nan"), dtype=torch.float32, device="cuda")
    Vd = torch.full((cols, l), float("nan"), dtype=torch.float32, device="cuda")
    sd = torch.full((l,), float("nan"), dtype=torch.float32, device="cuda")
    nbytes = M.mdbf_msvid_workspace_bytes(rows, cols, l)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    M.mdbf_project_fixed_mask(Zd.data_ptr(), Sd.data_ptr(), rows, cols, l, n_iter, Qd.data_ptr(), Ud.data_ptr(), Vd.data_ptr(), sd.data_ptr(),
                              ws.data_ptr(), nbytes, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return Ud.cpu().numpy().astype(np.float64), Vd.cpu().numpy().astype(np.float64), sd.cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("shape,l", [((300, 517), 4), ((1024, 768), 16), ((129, 33), 1), ((64, 2000), 8), ((700, 900), 32)])
def test_projection_under_a_given_mask(shape, l):
    """Theorem 1 with a mask that is NOT the sign of Z: the envelope S (.) Z has entries of both signs and no dominant
    direction; the error of the projection is bounded below by Eq. rankl-error and the iteration ends close to it."""
    rows, cols = shape
    Z = inputs.make_factor_matrix(rows, cols, seed=9, special_values=False)
    S = inputs.make_signs(rows, cols, seed=21, stream="S_A")
    P_ref, sv = orc.project_fixed_mask(S, Z, l)
    tail = np.sqrt(np.sum(sv[l:] ** 2))
    U, V, s = run_projection(Z, S, l, n_iter=12)
    assert np.all(np.isfinite(U)) and np.all(np.isfinite(V))
    assert np.all(s <= sv[:l] * (1 + 2e-5)) and np.all(s >= 0.75 * sv[:l])
    P = S * (U @ V.T)
    err = np.linalg.norm(Z.astype(np.float64) - P)
    assert abs(np.linalg.norm(Z.astype(np.float64) - P_ref) - tail) <= 1e-9 * sv[0]      # the oracle attains the bound
    assert tail * (1 - 1e-5) <= err <= tail * 1.02
    # the envelope error is the same number (Eq. envelope-isometry)
    assert abs(np.linalg.norm(S * Z.astype(np.float64) - U @ V.T) - err) <= 1e-9 * sv[0]


def test_projection_with_the_matrix_own_mask_is_msvid():
    Z = inputs.make_factor_matrix(257, 390, seed=10)
    S = np.where(Z >= 0, 1, -1).astype(np.int8)
    _, U1, V1, s1 = run_msvid(Z, 8, n_iter=5)
    U2, V2, s2 = run_projection(Z, S, 8, n_iter=5)
    np.testing.assert_array_equal(s1, s2)                    # the same kernels on the same envelope: the same bits
    np.testing.assert_array_equal(U1, U2)
    np.testing.assert_array_equal(V1, V2)


def test_msvid_of_both_factors_makes_a_layer():
    """Eq. mesvid-init-compact from given balanced factors: MSVID_l of U0 (d_out x k) and of V0^T (k x d_in) on the GPU,
    the two masks and envelopes packed into a layer, and that layer's dense reconstruction and forward compared with
    the oracle's - whose own MSVID (exact SVD) sets the approximation error the GPU initialisation has to come close to."""
    d_out, d_in, k, l = 384, 320, 128, 8
    rng = np.random.default_rng(44)
    W = (rng.standard_normal((d_out, 48)) @ rng.standard_normal((48, d_in)) / 7 + 0.3 * rng.standard_normal((d_out, d_in)))
    Uw, sw, Vwt = np.linalg.svd(W, full_matrices=False)
    U0 = (Uw[:, :k] * np.sqrt(sw[:k])).astype(np.float32)                  # Eq. mesvid-balanced, given as inputs
    V0t = (np.sqrt(sw[:k])[:, None] * Vwt[:k]).astype(np.float32)
    W_R = U0.astype(np.float64) @ V0t.astype(np.float64)
    SpA, UA, VA, _ = run_msvid(U0, l, n_iter=12)
    SpB, UB, VB, _ = run_msvid(V0t, l, n_iter=12)
    S_A, S_B = orc.unpack_signs(SpA, k), orc.unpack_signs(SpB, d_in)
    # the same construction in the oracle (exact truncated SVDs)
    So_A, Uo_A, Vo_A = orc.msvid(U0, l)
    So_B, Uo_B, Vo_B = orc.msvid(V0t, l)
    np.testing.assert_array_equal(S_A, So_A)
    np.testing.assert_array_equal(S_B, So_B)
    W_gpu_init = orc.reconstruct(S_A, S_B, UA, VA, UB, VB)
    W_orc_init = orc.reconstruct(So_A, So_B, Uo_A, Vo_A, Uo_B, Vo_B)
    e_gpu = np.linalg.norm(W_R - W_gpu_init) / np.linalg.norm(W_R)
    e_orc = np.linalg.norm(W_R - W_orc_init) / np.linalg.norm(W_R)
    assert e_gpu <= e_orc * 1.03                                            # the initialisation is as good as the exact one, within 3 %
    # the factors as a layer of the library (fp32 envelopes: no storage rounding in the way)
    h = M.mdbf_pack(d_out, d_in, k, l, M.F32, 4, S_A, S_B, *[np.ascontiguousarray(a, dtype=np.float32) for a in (UA, VA, UB, VB)])
    try:
        Wd = torch.empty((d_out, d_in), dtype=torch.float32, device="cuda")
        M.mdbf_reconstruct(h, Wd.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert orc.rel_frobenius(Wd.cpu().numpy(), W_gpu_init) <= 1e-6
        x = rng.standard_normal((4, d_in)).astype(np.float32)
        xd = torch.from_numpy(x).cuda()
        yd = torch.empty((4, d_out), dtype=torch.float32, device="cuda")
        M.mdbf_linear_forward(h, xd.data_ptr(), yd.data_ptr(), 4, M.F32, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        ref = (W_gpu_init @ x.T.astype(np.float64)).T
        assert orc.rel_frobenius(yd.cpu().numpy(), ref) <= 1e-5
    finally:
        M.mdbf_destroy(h)


def test_argument_errors():
    Z = torch.zeros((8, 8), dtype=torch.float32, device="cuda")
    Q = torch.ones((8, 2), dtype=torch.float32, device="cuda")
    S = torch.zeros((8, 1), dtype=torch.int32, device="cuda")
    U = torch.zeros((8, 2), dtype=torch.float32, device="cuda")
    s = torch.zeros((2,), dtype=torch.float32, device="cuda")
    nbytes = M.mdbf_msvid_workspace_bytes(8, 8, 2)
    ws = torch.zeros(nbytes + 256, dtype=torch.uint8, device="cuda")
    args = lambda: [Z.data_ptr(), 8, 8, 2, 2, Q.data_ptr(), S.data_ptr(), U.data_ptr(), U.data_ptr(), s.data_ptr(), ws.data_ptr(), nbytes]
    for pos, val, status in ((0, 0, M.ERR_INVALID_ARG), (1, 0, M.ERR_SHAPE), (3, 0, M.ERR_SHAPE), (3, 33, M.ERR_SHAPE),
                             (3, 9, M.ERR_SHAPE), (4, 0, M.ERR_SHAPE), (10, 0, M.ERR_INVALID_ARG), (11, nbytes - 1, M.ERR_INVALID_ARG),
                             (10, ws.data_ptr() + 4, M.ERR_INVALID_ARG)):
        a = args()
        a[pos] = val
        with pytest.raises(M.MdbfError) as e:
            M.mdbf_msvid(*a)
        assert e.value.status == status
    with pytest.raises(M.MdbfError):
        M.mdbf_msvid_workspace_bytes(8, 8, 9)
    M.mdbf_msvid(*args())                                    # and the same arguments untouched go through
    torch.cuda.synchronize()
