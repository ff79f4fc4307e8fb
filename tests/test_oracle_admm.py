"""Pins of the oracle's ADMM factor update (Eq. admm-U-tilde, Eq. admm-U-prox, Eq. admm-U-dual) against what the
paper and the mathematics fix, and planted mistakes that the pins must notice."""
import types

import numpy as np
import pytest

from oracle import mdbf_oracle as orc


def _problem(seed=0, N=14, M=11, R=6):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((N, M)), rng.standard_normal((M, R)), rng.standard_normal((N, R)),
            0.3 * rng.standard_normal((N, R)))


def pin_scalar_instance_by_hand(o):
    """N = M = R = l = 1: W = 3, V = 2, U = 1, Lam = 1/2, rho = 1.  U_tilde = (3*2 + (1 - 1/2)) / (2*2 + 1) = 1.3;
    MSVID_1 of a scalar is the scalar: U = 1.3 + 0.5 = 1.8; Lam = 0.5 + 1.3 - 1.8 = 0."""
    U, Lam, tildes, masks = o.admm_factor_update([[3.0]], [[2.0]], [[1.0]], [[0.5]], 1.0, 1, 1)
    assert abs(tildes[0][0, 0] - 1.3) < 1e-12
    assert abs(U[0, 0] - 1.8) < 1e-12
    assert abs(Lam[0, 0]) < 1e-12
    assert masks[0][0, 0] == 1
    # a second inner iteration from there: U_tilde = (6 + 1.8) / 5 = 1.56, U = 1.56, Lam = 0
    U2, Lam2, tildes2, _ = o.admm_factor_update([[3.0]], [[2.0]], [[1.0]], [[0.5]], 1.0, 1, 2)
    assert abs(tildes2[1][0, 0] - 1.56) < 1e-12 and abs(U2[0, 0] - 1.56) < 1e-12 and abs(Lam2[0, 0]) < 1e-12
    # negative values keep their sign through MSVID: W = -3 mirrors everything
    U3, _, tildes3, masks3 = o.admm_factor_update([[-3.0]], [[2.0]], [[-1.0]], [[-0.5]], 1.0, 1, 1)
    assert abs(tildes3[0][0, 0] + 1.3) < 1e-12 and abs(U3[0, 0] + 1.8) < 1e-12 and masks3[0][0, 0] == -1


def pin_least_squares_step_is_the_minimiser(o):
    """U_tilde minimises f(X) = 1/2 ||W - X V^T||^2 + rho/2 ||X - (U - Lam)||^2: the gradient vanishes there and no
    perturbed point does better."""
    W, V, U, Lam = _problem(1)
    rho = 0.7
    _, _, tildes, _ = o.admm_factor_update(W, V, U, Lam, rho, 2, 1)
    X = tildes[0]

    def f(X):
        return 0.5 * np.sum((W - X @ V.T) ** 2) + 0.5 * rho * np.sum((X - (U - Lam)) ** 2)
    grad = -(W - X @ V.T) @ V + rho * (X - (U - Lam))
    assert np.max(np.abs(grad)) < 1e-9
    rng = np.random.default_rng(5)
    for _ in range(20):
        assert f(X) <= f(X + 1e-3 * rng.standard_normal(X.shape))


def pin_large_penalty_limit(o):
    """rho -> infinity pins U_tilde to U - Lam."""
    W, V, U, Lam = _problem(2)
    _, _, tildes, _ = o.admm_factor_update(W, V, U, Lam, 1e12, 2, 1)
    assert np.max(np.abs(tildes[0] - (U - Lam))) < 1e-8


def pin_fixed_point_at_a_representable_factor(o):
    """W = U V^T with U in F_l(S) and Lam = 0: the least-squares step returns U, MSVID_l leaves it, Lam stays 0."""
    rng = np.random.default_rng(3)
    N, M, R, l = 12, 10, 5, 2
    S = np.where(rng.random((N, R)) < 0.5, -1.0, 1.0)
    U = S * (np.abs(rng.standard_normal((N, l))) @ np.abs(rng.standard_normal((R, l))).T)      # positive envelope of rank l
    V = rng.standard_normal((M, R))
    Un, Ln, tildes, masks = o.admm_factor_update(U @ V.T, V, U, np.zeros_like(U), 0.5, l, 3)
    assert np.max(np.abs(Un - U)) < 1e-9 and np.max(np.abs(Ln)) < 1e-9
    assert np.array_equal(masks[-1], S.astype(np.int8))


def pin_result_has_the_format_and_the_dual_balances(o):
    """The new U carries an envelope of rank <= l under its own mask (Eq. me-dbf-envelope-rank), and the three iterates
    close the loop: U_tilde + Lam_old = U + Lam_new."""
    W, V, U, Lam = _problem(4)
    l = 2
    Un, Ln, tildes, masks = o.admm_factor_update(W, V, U, Lam, 0.9, l, 1)
    sv = np.linalg.svd(masks[0] * Un, compute_uv=False)
    assert sv[l] < 1e-9 * sv[0]          # (the truncated envelope itself may have entries below zero)
    assert np.max(np.abs(tildes[0] + Lam - Un - Ln)) < 1e-12
    # the step is MSVID's: no matrix with that mask and rank-l envelope is closer to U_tilde + Lam (Theorem 1)
    Z = tildes[0] + Lam
    tail = np.sqrt(np.sum(np.linalg.svd(np.abs(Z), compute_uv=False)[l:] ** 2))
    assert abs(np.linalg.norm(Z - Un) - tail) < 1e-9


def pin_transposed_problem_updates_the_other_factor(o):
    """The V update is the same function on W^T with the roles of the factors exchanged: at rho -> 0+ and l = R = full
    rank it returns the least-squares V for the given U."""
    rng = np.random.default_rng(6)
    N, M, R = 9, 8, 3
    U = rng.standard_normal((N, R))
    W = rng.standard_normal((N, M))
    _, _, tildes, _ = o.admm_factor_update(W.T, U, np.zeros((M, R)), np.zeros((M, R)), 1e-12, R, 1)
    V_ls = np.linalg.lstsq(U, W, rcond=None)[0].T
    assert np.max(np.abs(tildes[0] - V_ls)) < 1e-6


ADMM_PINS = [pin_scalar_instance_by_hand, pin_least_squares_step_is_the_minimiser, pin_large_penalty_limit,
             pin_fixed_point_at_a_representable_factor, pin_result_has_the_format_and_the_dual_balances,
             pin_transposed_problem_updates_the_other_factor]


@pytest.mark.parametrize("pin", ADMM_PINS, ids=lambda p: p.__name__)
def test_admm_pin(pin):
    pin(orc)


def _mutants():
    real = orc

    def variant(prox_sign=1.0, dual_sign=1.0, ridge=True, diff_sign=-1.0, solve_side="right"):
        def f(W, V, U, Lam, rho, l, n_inner=1):
            W, V, U, Lam = (np.asarray(a, dtype=np.float64) for a in (W, V, U, Lam))
            R = V.shape[1]
            G = V.T @ V + (rho if ridge else 0.0) * np.eye(R)
            tildes, masks = [], []
            for _ in range(n_inner):
                rhs = W @ V + rho * (U + diff_sign * Lam)
                Ut = np.linalg.solve(G, rhs.T).T if solve_side == "right" else np.linalg.solve(G.T + np.triu(G, 1) * 0.5, rhs.T).T
                S, Ul, Vl = real.msvid(Ut + prox_sign * Lam, l)
                U = S * (Ul @ Vl.T)
                Lam = Lam + dual_sign * (Ut - U)
                tildes.append(Ut)
                masks.append(S)
            return U, Lam, tildes, masks
        return types.SimpleNamespace(admm_factor_update=f, msvid=real.msvid)

    def no_prox(W, V, U, Lam, rho, l, n_inner=1):
        Un, Ln, t, m = real.admm_factor_update(W, V, U, Lam, rho, l, n_inner)
        return t[-1] + (np.asarray(Lam, dtype=np.float64) if n_inner == 1 else 0), Ln, t, m
    return {
        "dual added in the least-squares step": variant(diff_sign=+1.0),
        "dual subtracted in the prox step": variant(prox_sign=-1.0),
        "dual update with the wrong sign": variant(dual_sign=-1.0),
        "ridge term dropped": variant(ridge=False),
        "asymmetric system solved": variant(solve_side="other"),
        "prox step skipped": types.SimpleNamespace(admm_factor_update=no_prox),
    }


@pytest.mark.parametrize("name", sorted(_mutants().keys()))
def test_planted_mistakes_in_the_admm_update_are_caught(name):
    mutant = _mutants()[name]
    caught = []
    for pin in ADMM_PINS:
        try:
            pin(mutant)
        except (AssertionError, ValueError, IndexError, np.linalg.LinAlgError):
            caught.append(pin.__name__)
    assert caught, f"no pin notices the planted mistake: {name}"
