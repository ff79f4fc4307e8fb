"""ADMM refinement of a factor on the GPU (mdbf_admm_factor_update; Eq. admm-U-tilde, Eq. admm-U-prox, Eq. admm-U-dual)
against the oracle.  The least-squares iterate is compared element by element; the prox step is MSVID computed by subspace
iteration, so what follows it is compared through what is unique: the sign mask away from zero, Theorem 1's error, the
objective, and the identities that tie the iterates together."""
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


def problem(N, Mc, R, seed):
    W = inputs.make_factor_matrix(N, Mc, seed, special_values=False)
    V = inputs.make_factor_matrix(Mc, R, seed + 1, special_values=False)
    U = inputs.make_factor_matrix(N, R, seed + 2, special_values=False)
    Lam = (0.1 * inputs.make_factor_matrix(N, R, seed + 3, special_values=False)).astype(np.float32)
    return W, V, U, Lam


def run_update(W, V, U, Lam, rho, l, n_inner, n_iter, transpose=False, want_tilde=True):
    Wop = W.T if transpose else W
    N, R = U.shape
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    Wd, Vd, Ud, Ld = dev(W), dev(V), dev(U), dev(Lam)
    Qd = dev(inputs.make_start_block(R, l, 17))
    nwords = (R + 31) // 32
    Sd = torch.zeros((N, nwords), dtype=torch.int32, device="cuda")
    Uld = torch.zeros((N, l), dtype=torch.float32, device="cuda")
    Vld = torch.zeros((R, l), dtype=torch.float32, device="cuda")
    sd = torch.zeros((l,), dtype=torch.float32, device="cuda")
    Td = torch.zeros((N, R), dtype=torch.float32, device="cuda") if want_tilde else None
    nbytes = M.mdbf_admm_workspace_bytes(N, Wop.shape[1], R, l)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    M.mdbf_admm_factor_update(Wd.data_ptr(), W.shape[0], W.shape[1], transpose, Vd.data_ptr(), R, Ud.data_ptr(), Ld.data_ptr(), rho, l,
                              n_inner, n_iter, Qd.data_ptr(), Sd.data_ptr(), Uld.data_ptr(), Vld.data_ptr(), sd.data_ptr(),
                              Td.data_ptr() if want_tilde else None, ws.data_ptr(), nbytes, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    f64 = lambda t: t.cpu().numpy().astype(np.float64)
    assert Wop.shape[0] == N
    return dict(U=f64(Ud), Lam=f64(Ld), S=Sd.cpu().numpy().view(np.uint32), Ul=f64(Uld), Vl=f64(Vld), sigma=f64(sd),
                tilde=f64(Td) if want_tilde else None)


@pytest.mark.parametrize("N,Mc,R,l,transpose", [(300, 260, 64, 4, False), (515, 384, 128, 16, False), (260, 300, 64, 8, True),
                                                (200, 150, 50, 4, False), (130, 700, 36, 32, False)])
def test_one_inner_iteration(N, Mc, R, l, transpose):
    Wop, V, U, Lam = problem(N, Mc, R, seed=31)
    W = np.ascontiguousarray(Wop.T) if transpose else Wop                  # what the caller stores; op(W) = Wop either way
    rho = 0.05 * float(np.sum(V.astype(np.float64) ** 2)) / R
    g = run_update(W, V, U, Lam, rho, l, 1, 10, transpose)
    Uo, Lo, tildes, masks = orc.admm_factor_update(Wop, V, U, Lam, rho, l, 1)
    # the least-squares iterate: fp32 products and an fp32 Cholesky solve against fp64
    scale = np.max(np.abs(tildes[0]))
    assert np.max(np.abs(g["tilde"] - tildes[0])) <= 2e-4 * scale
    # the mask of U_tilde + Lam: exact wherever the argument is not within rounding of zero
    Zo = tildes[0] + Lam.astype(np.float64)
    Sg = orc.unpack_signs(g["S"], R)
    clear = np.abs(Zo) > 5e-4 * scale                  # more than twice the tolerance on U_tilde
    assert clear.mean() > 0.9
    np.testing.assert_array_equal(Sg[clear], masks[0][clear])
    # the compact form is the dense one
    np.testing.assert_allclose(g["U"], Sg * (g["Ul"] @ g["Vl"].T), atol=2e-5 * scale)
    # prox step: Theorem 1's error is a lower bound for any matrix of the format, and the iteration comes close to it
    Zg = g["tilde"] + Lam.astype(np.float64)
    tail = np.sqrt(np.sum(np.linalg.svd(np.abs(Zg), compute_uv=False)[l:] ** 2))
    err = np.linalg.norm(Zg - g["U"])
    assert tail * (1 - 1e-4) <= err <= tail * 1.02 + 1e-5 * scale
    # the dual closes the loop with the GPU's own iterates
    np.testing.assert_allclose(g["Lam"], Lam.astype(np.float64) + g["tilde"] - g["U"], atol=2e-5 * scale)
    # and the objective is the oracle's
    obj_g = np.linalg.norm(Wop.astype(np.float64) - g["U"] @ V.astype(np.float64).T)
    obj_o = np.linalg.norm(Wop.astype(np.float64) - Uo @ V.astype(np.float64).T)
    assert abs(obj_g - obj_o) <= 0.01 * obj_o


@pytest.mark.parametrize("trial", range(12))
def test_random_ragged_shapes(trial):
    """Sizes drawn at random, none a multiple of a tile: the products' tails (rows, columns, contraction indices, an odd number
    of 128-column tiles), both orientations of W."""
    rng = np.random.default_rng(900 + trial)
    N, Mc = int(rng.integers(2, 900)), int(rng.integers(2, 900))
    R = int(min(rng.integers(1, min(N, Mc) + 1), 600))
    l = int(min(rng.choice([1, 2, 4, 8, 16, 32]), R, N))
    transpose = bool(trial % 2)
    Wop, V, U, Lam = problem(N, Mc, R, seed=500 + trial)
    W = np.ascontiguousarray(Wop.T) if transpose else Wop
    rho = float(np.sum(V.astype(np.float64) ** 2)) / R
    g = run_update(W, V, U, Lam, rho, l, 1, 6, transpose)
    _, _, tildes, _ = orc.admm_factor_update(Wop, V, U, Lam, rho, l, 1)
    scale = np.max(np.abs(tildes[0]))
    assert np.max(np.abs(g["tilde"] - tildes[0])) <= 2e-5 * scale
    np.testing.assert_allclose(g["Lam"], Lam.astype(np.float64) + g["tilde"] - g["U"], atol=2e-5 * scale)
    assert np.all(np.isfinite(g["U"])) and np.all(np.isfinite(g["sigma"]))


def test_several_inner_iterations_follow_the_oracle():
    W, V, U, Lam = problem(400, 320, 96, seed=41)
    rho = float(np.sum(V.astype(np.float64) ** 2)) / 96
    l = 8
    for n_inner in (2, 4):
        g = run_update(W, V, U, Lam, rho, l, n_inner, 10, want_tilde=False)
        Uo, Lo, tildes, masks = orc.admm_factor_update(W, V, U, Lam, rho, l, n_inner)
        assert np.all(np.isfinite(g["U"])) and np.all(np.isfinite(g["Lam"]))
        obj_g = np.linalg.norm(W.astype(np.float64) - g["U"] @ V.astype(np.float64).T)
        obj_o = np.linalg.norm(W.astype(np.float64) - Uo @ V.astype(np.float64).T)
        assert abs(obj_g - obj_o) <= 0.02 * obj_o
        assert abs(np.linalg.norm(g["Lam"]) - np.linalg.norm(Lo)) <= 0.05 * np.linalg.norm(Lo) + 1e-6
        agree = np.mean(orc.unpack_signs(g["S"], 96) == masks[-1])
        assert agree > 0.9                                # entries near zero may fall either way; most of the mask is the oracle's


def test_refinement_of_an_msvid_initialisation_lowers_the_objective():
    """Eq. mesvid-init-compact followed by alternating updates of both factors (the paper's use of the scheme): with the penalty
    at the scale of V^T V's diagonal the reconstruction error of W_hat = U V^T falls below the initialisation's, and the GPU's
    run ends where the oracle's does."""
    rng_W = inputs.make_factor_matrix(256, 192, 51, special_values=False).astype(np.float64)
    R, l = 64, 4
    Uu, s, Vt = np.linalg.svd(rng_W, full_matrices=False)
    U0, V0 = Uu[:, :R] * np.sqrt(s[:R]), Vt[:R].T * np.sqrt(s[:R])                   # balanced factors (Eq. mesvid-balanced)
    SU, Au, Bu = orc.msvid(U0, l)
    SV, Av, Bv = orc.msvid(V0, l)
    U, V = SU * (Au @ Bu.T), SV * (Av @ Bv.T)
    W = rng_W.astype(np.float32)
    start = np.linalg.norm(rng_W - U @ V.T)
    rho = float(np.sum(V ** 2)) / R
    Uo, Vo = U.copy(), V.copy()
    LamU, LamV = np.zeros_like(U), np.zeros_like(V)
    LoU, LoV = np.zeros_like(U), np.zeros_like(V)
    for _ in range(3):
        g = run_update(W, V, U, LamU, rho, l, 3, 10, want_tilde=False)
        U, LamU = g["U"], g["Lam"]
        g = run_update(W, U, V, LamV, rho, l, 3, 10, transpose=True, want_tilde=False)
        V, LamV = g["U"], g["Lam"]
        Uo, LoU, _, _ = orc.admm_factor_update(rng_W, Vo, Uo, LoU, rho, l, 3)
        Vo, LoV, _, _ = orc.admm_factor_update(rng_W.T, Uo, Vo, LoV, rho, l, 3)
    end, end_o = np.linalg.norm(rng_W - U @ V.T), np.linalg.norm(rng_W - Uo @ Vo.T)
    assert end_o < 0.9 * start                                  # the scheme does refine (oracle)
    assert np.isfinite(end) and abs(end - end_o) <= 0.03 * end_o


def test_failed_allocation_of_the_solver_scratch_is_reported_and_leaves_the_library_usable():
    """The factorisation's scratch is the one allocation of this call (first call of a host thread).  A fresh thread with the
    library's allocation-failure hook armed gets an error, not a fault; the same thread's next call succeeds and matches a
    run in the main thread."""
    import threading
    W, V, U, Lam = problem(128, 96, 32, seed=61)
    rho = float(np.sum(V.astype(np.float64) ** 2)) / 32
    ref = run_update(W, V, U, Lam, rho, 4, 1, 6)
    out = {}

    def worker():
        torch.cuda.set_device(0)
        M.mdbf_debug_fail_alloc(1)
        try:
            run_update(W, V, U, Lam, rho, 4, 1, 6)
            out["first"] = "no error"
        except M.MdbfError as e:
            out["first"] = str(e)
        finally:
            M.mdbf_debug_fail_alloc(0)
        out["second"] = run_update(W, V, U, Lam, rho, 4, 1, 6)
    t = threading.Thread(target=worker)
    t.start()
    t.join()
    assert "out of device memory" in out["first"], out["first"]
    np.testing.assert_array_equal(out["second"]["tilde"], ref["tilde"])
    np.testing.assert_array_equal(out["second"]["S"], ref["S"])


def test_argument_errors():
    W, V, U, Lam = problem(64, 48, 32, seed=3)
    with pytest.raises(M.MdbfError):
        run_update(W, V, U, Lam, 0.0, 4, 1, 4)
    with pytest.raises(M.MdbfError):
        run_update(W, V, U, Lam, 1.0, 33, 1, 4)
    with pytest.raises(M.MdbfError):
        M.mdbf_admm_workspace_bytes(0, 48, 32, 4)
    d = torch.zeros(16, device="cuda")
    with pytest.raises(M.MdbfError):           # workspace too small
        M.mdbf_admm_factor_update(d.data_ptr(), 64, 48, False, d.data_ptr(), 32, d.data_ptr(), d.data_ptr(), 1.0, 4, 1, 4, d.data_ptr(),
                                  d.data_ptr(), d.data_ptr(), d.data_ptr(), d.data_ptr(), None, d.data_ptr(), 64, 0)


def test_bench_size_update_on_sampled_rows():
    """The shape bench.py times (N = M = 8192, R = 3712, l = 16): the least-squares iterate of sampled rows against the
    definition evaluated in fp64 (Eq. admm-U-tilde row by row: a row of U_tilde depends on its rows of W, U and Lambda and
    on V only), the mask of those rows, and the identities that tie the outputs together."""
    N, Mc, R, l = 8192, 8192, 3712, 16
    W, V, U = (inputs.make_factor_matrix(a, b, seed=60 + i, special_values=False) for i, (a, b) in enumerate([(N, Mc), (Mc, R), (N, R)]))
    Lam = (0.1 * inputs.make_factor_matrix(N, R, seed=63, special_values=False)).astype(np.float32)
    V64 = V.astype(np.float64)
    rho = float(np.sum(V64 ** 2)) / R
    g = run_update(W, V, U, Lam, rho, l, 1, 4)
    rows = np.random.default_rng(5).choice(N, size=24, replace=False)
    G = V64.T @ V64 + rho * np.eye(R)
    rhs = W[rows].astype(np.float64) @ V64 + rho * (U[rows].astype(np.float64) - Lam[rows].astype(np.float64))
    tilde_ref = np.linalg.solve(G, rhs.T).T
    scale = np.max(np.abs(tilde_ref))
    # 3e-6 measured; one accumulator over all 8192 contraction indices would be at 6e-5 (the tensor core's accumulation is not
    # rounded to nearest), which is why the product kernel accumulates in chunks
    assert np.max(np.abs(g["tilde"][rows] - tilde_ref)) <= 1.5e-5 * scale
    Z = tilde_ref + Lam[rows].astype(np.float64)
    Sg = orc.unpack_signs(g["S"][rows], R)
    clear = np.abs(Z) > 5e-4 * scale
    np.testing.assert_array_equal(Sg[clear], np.where(Z >= 0, 1, -1)[clear])
    np.testing.assert_allclose(g["U"][rows], Sg * (g["Ul"][rows] @ g["Vl"].T), atol=2e-5 * scale)
    np.testing.assert_allclose(g["Lam"][rows], Lam[rows].astype(np.float64) + g["tilde"][rows] - g["U"][rows], atol=2e-5 * scale)
    assert np.all(np.isfinite(g["sigma"])) and np.all(np.diff(g["sigma"]) <= 1e-6 * g["sigma"][0])
