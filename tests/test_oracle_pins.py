"""Pins for the CPU oracle: what the paper and the mathematics fix, none of it
computed by the oracle's own formula.  CPU only.

Each `pin_*` takes an oracle-like namespace so that the same checks can be run
against deliberately broken copies (test_planted_mistakes_are_caught): a
plausible mistake anywhere in the oracle must fail at least one pin.
"""
import itertools
import json
import os
import types

import numpy as np
import pytest

from oracle import mdbf_oracle as real
from oracle import loops

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_layer(rng, d_out, d_in, k, l):
    S_A = rng.choice(np.array([-1, 1], dtype=np.int8), size=(d_out, k))
    S_B = rng.choice(np.array([-1, 1], dtype=np.int8), size=(k, d_in))
    U_A = rng.standard_normal((d_out, l))
    V_A = rng.standard_normal((k, l))
    U_B = rng.standard_normal((k, l))
    V_B = rng.standard_normal((d_in, l))
    return S_A, S_B, U_A, V_A, U_B, V_B


# --------------------------------------------------------------------- pins
def pin_worked_example(o):
    """Hand-worked numbers (tests/golden/worked_example.json)."""
    g = json.load(open(os.path.join(GOLDEN, "worked_example.json")))
    a = {k: np.array(v) for k, v in g.items() if not k.startswith("_")}
    lay = (a["S_A"], a["S_B"], a["U_A"], a["V_A"], a["U_B"], a["V_B"])
    np.testing.assert_allclose(o.envelope(a["U_A"], a["V_A"]), a["E_A"], atol=1e-12)
    np.testing.assert_allclose(o.modulated_factor(a["S_A"], a["U_A"], a["V_A"]), a["U_hat"], atol=1e-12)
    np.testing.assert_allclose(o.modulated_factor(a["S_B"], a["U_B"], a["V_B"]), a["V_hat_T"], atol=1e-12)
    np.testing.assert_allclose(o.reconstruct(*lay), a["W_hat"], atol=1e-12)
    np.testing.assert_allclose(o.forward(*lay, a["x"]), a["y"], atol=1e-12)
    y, z = o.forward_staged(*lay, a["x"])
    np.testing.assert_allclose(z, a["z"], atol=1e-12)
    np.testing.assert_allclose(y, a["y"], atol=1e-12)
    np.testing.assert_allclose(o.reconstruct_rows([1], *lay), a["W_hat"][1:2], atol=1e-12)


def pin_sum_of_dbf(o):
    """Eq. me-dbf-sum: W_hat = sum_t sum_s D_{a^(t)} S_a D_{q^(t) (.) g^(s)} S_b^T D_{b^(s)},
    written with explicit diagonal matrices."""
    rng = np.random.default_rng(11)
    for (d_out, d_in, k, l) in [(5, 7, 6, 3), (9, 4, 3, 2), (6, 6, 8, 1)]:
        S_A, S_B, U_A, V_A, U_B, V_B = rand_layer(rng, d_out, d_in, k, l)
        W = np.zeros((d_out, d_in))
        for t in range(l):
            for s in range(l):
                W += (np.diag(U_A[:, t]) @ S_A.astype(float) @ np.diag(V_A[:, t] * U_B[:, s])
                      @ S_B.astype(float) @ np.diag(V_B[:, s]))
        got = o.reconstruct(S_A, S_B, U_A, V_A, U_B, V_B)
        assert real.rel_frobenius(got, W) < 1e-13
        X = rng.standard_normal((d_in, 3))
        assert real.rel_frobenius(o.forward(S_A, S_B, U_A, V_A, U_B, V_B, X), W @ X) < 1e-13
        Y, Z = o.forward_staged(S_A, S_B, U_A, V_A, U_B, V_B, X)
        assert real.rel_frobenius(Y, W @ X) < 1e-13
        rows = [d_out - 1, 0]
        assert real.rel_frobenius(o.reconstruct_rows(rows, S_A, S_B, U_A, V_A, U_B, V_B), W[rows]) < 1e-13


def pin_l1_is_dbf(o):
    """l = 1 reduces to D_a S_a D_m S_b^T D_b with m = q (.) g (Eq. dbf-basis)."""
    rng = np.random.default_rng(12)
    d_out, d_in, k = 6, 5, 7
    S_A, S_B, U_A, V_A, U_B, V_B = rand_layer(rng, d_out, d_in, k, 1)
    a, q, g, b = U_A[:, 0], V_A[:, 0], U_B[:, 0], V_B[:, 0]
    W = np.zeros((d_out, d_in))
    for n in range(d_out):
        for i in range(d_in):
            W[n, i] = a[n] * sum(S_A[n, j] * q[j] * g[j] * S_B[j, i] for j in range(k)) * b[i]
    assert real.rel_frobenius(o.reconstruct(S_A, S_B, U_A, V_A, U_B, V_B), W) < 1e-13
    x = rng.standard_normal(d_in)
    # Eq. DBF-inference-form, transposed: y = a (.) (S_a (m (.) (S_b^T (b (.) x))))
    y = a * (S_A.astype(float) @ ((q * g) * (S_B.astype(float) @ (b * x))))
    np.testing.assert_allclose(o.forward(S_A, S_B, U_A, V_A, U_B, V_B, x), y, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(o.forward_staged(S_A, S_B, U_A, V_A, U_B, V_B, x)[0], y, rtol=1e-12, atol=1e-12)


def pin_all_plus_signs(o):
    """All-(+1) signs: W_hat is the plain low-rank product (U_A V_A^T)(U_B V_B^T)."""
    rng = np.random.default_rng(13)
    d_out, d_in, k, l = 7, 9, 5, 3
    _, _, U_A, V_A, U_B, V_B = rand_layer(rng, d_out, d_in, k, l)
    S_A = np.ones((d_out, k), dtype=np.int8)
    S_B = np.ones((k, d_in), dtype=np.int8)
    W = np.linalg.multi_dot([U_A, V_A.T, U_B, V_B.T])
    assert real.rel_frobenius(o.reconstruct(S_A, S_B, U_A, V_A, U_B, V_B), W) < 1e-13


def pin_gauge_and_flips(o):
    """Column j of S_A and row j of S_B flipped together leave W_hat unchanged
    (column-sign absorption, end of Section 4.2); flipping column j of S_A alone
    equals negating row j of V_A; flipping row n of S_A negates row n of W_hat
    only if done on the whole row."""
    rng = np.random.default_rng(14)
    d_out, d_in, k, l = 6, 8, 5, 2
    S_A, S_B, U_A, V_A, U_B, V_B = rand_layer(rng, d_out, d_in, k, l)
    W = o.reconstruct(S_A, S_B, U_A, V_A, U_B, V_B)
    j = 3
    S_A2, S_B2 = S_A.copy(), S_B.copy()
    S_A2[:, j] *= -1
    S_B2[j, :] *= -1
    np.testing.assert_allclose(o.reconstruct(S_A2, S_B2, U_A, V_A, U_B, V_B), W, atol=1e-12)
    V_A2 = V_A.copy()
    V_A2[j, :] *= -1
    np.testing.assert_allclose(o.reconstruct(S_A2, S_B, U_A, V_A, U_B, V_B),
                               o.reconstruct(S_A, S_B, U_A, V_A2, U_B, V_B), atol=1e-12)
    S_A3 = S_A.copy()
    S_A3[2, :] *= -1
    W3 = o.reconstruct(S_A3, S_B, U_A, V_A, U_B, V_B)
    np.testing.assert_allclose(W3[2], -W[2], atol=1e-12)
    np.testing.assert_allclose(np.delete(W3, 2, 0), np.delete(W, 2, 0), atol=1e-12)
    # a single sign flip changes W_hat by the rank-one term it multiplies
    S_B4 = S_B.copy()
    S_B4[1, 4] *= -1
    dW = o.reconstruct(S_A, S_B4, U_A, V_A, U_B, V_B) - W
    E_B = U_B @ V_B.T
    U_hat = S_A * (U_A @ V_A.T)
    expect = np.zeros_like(W)
    expect[:, 4] = U_hat[:, 1] * (-2.0 * S_B[1, 4] * E_B[1, 4])
    np.testing.assert_allclose(dW, expect, atol=1e-12)


def pin_demodulation_and_isometry(o):
    """S (.) U_hat = A Q^T has rank <= l (Eq. me-dbf-envelope-rank);
    ||S (.) E||_F = ||E||_F (Lemma sign-mask isometry)."""
    rng = np.random.default_rng(15)
    p, q, l = 12, 10, 3
    S = rng.choice(np.array([-1, 1], dtype=np.int8), size=(p, q))
    U = rng.standard_normal((p, l))
    V = rng.standard_normal((q, l))
    F = o.modulated_factor(S, U, V)
    sv = np.linalg.svd(S * F, compute_uv=False)
    assert np.all(sv[l:] < 1e-12 * sv[0]) and sv[l - 1] > 1e-3 * sv[0]
    np.testing.assert_allclose(np.linalg.norm(F), np.linalg.norm(U @ V.T), rtol=1e-13)
    np.testing.assert_allclose(S * F, U @ V.T, atol=1e-12)
    # generic signs destroy the low rank of the modulated factor itself
    assert np.linalg.matrix_rank(F) > l


def pin_linearity_and_duality(o):
    """y is linear in x, columns are independent, and u^T (W v) = (W^T u)^T v where
    W^T is the same format with the factor roles swapped."""
    rng = np.random.default_rng(16)
    d_out, d_in, k, l = 7, 6, 4, 2
    lay = rand_layer(rng, d_out, d_in, k, l)
    S_A, S_B, U_A, V_A, U_B, V_B = lay
    X = rng.standard_normal((d_in, 4))
    Y = o.forward(*lay, X)
    for c in range(4):
        np.testing.assert_allclose(o.forward(*lay, X[:, c]), Y[:, c], atol=1e-12)
    np.testing.assert_allclose(o.forward(*lay, 2.0 * X[:, 0] - 3.0 * X[:, 1]),
                               2.0 * Y[:, 0] - 3.0 * Y[:, 1], atol=1e-11)
    u = rng.standard_normal(d_out)
    v = rng.standard_normal(d_in)
    layT = (S_B.T.copy(), S_A.T.copy(), V_B, U_B, V_A, U_A)
    lhs = u @ o.forward(*lay, v)
    rhs = o.forward(*layT, u) @ v
    np.testing.assert_allclose(lhs, rhs, rtol=1e-12)
    np.testing.assert_allclose(o.reconstruct(*layT), o.reconstruct(*lay).T, atol=1e-12)


def pin_metric(o):
    """Relative Frobenius error ||W - W_hat||_F / ||W||_F (Fig. 1 caption)."""
    A = np.array([[3.0, 0.0], [0.0, 4.0]])
    assert o.rel_frobenius(A, A) == 0.0
    assert o.rel_frobenius(np.zeros_like(A), A) == 1.0
    # ||(1,0;0,0)||_F / 5
    B = A.copy()
    B[0, 0] += 1.0
    np.testing.assert_allclose(o.rel_frobenius(B, A), 0.2, rtol=1e-15)
    np.testing.assert_allclose(o.rel_frobenius(A, 2 * A), 0.5, rtol=1e-15)   # normalised by the reference


def pin_packing(o):
    g = json.load(open(os.path.join(GOLDEN, "packing_examples.json")))
    for case in g["cases"]:
        S = np.array(case["signs"], dtype=np.int8)
        W = np.array(case["words"], dtype=np.uint32)
        np.testing.assert_array_equal(o.pack_signs(S), W)
        np.testing.assert_array_equal(o.unpack_signs(W, S.shape[1]), S)
    rng = np.random.default_rng(17)
    for rows, cols in [(3, 32), (4, 70), (1, 1), (5, 257), (2, 64)]:
        S = rng.choice(np.array([-1, 1], dtype=np.int8), size=(rows, cols))
        W = o.pack_signs(S)
        # independent library route: numpy.packbits, little-endian bit order, viewed as uint32
        pad = (-cols) % 32
        bits = np.pad((S == -1).astype(np.uint8), ((0, 0), (0, pad)))
        ref = np.packbits(bits, axis=1, bitorder="little").view("<u4")
        np.testing.assert_array_equal(W, ref)
        np.testing.assert_array_equal(loops.pack_signs(S), ref)
        np.testing.assert_array_equal(o.unpack_signs(W, cols), S)
    # every single-bit word and the extreme patterns
    for c in range(32):
        S = np.ones((1, 32), dtype=np.int8)
        S[0, c] = -1
        assert int(o.pack_signs(S)[0, 0]) == 1 << c
    assert int(o.pack_signs(-np.ones((1, 32), dtype=np.int8))[0, 0]) == 0xFFFFFFFF
    alt = np.where(np.arange(32) % 2 == 0, 1, -1).astype(np.int8)[None]
    assert int(o.pack_signs(alt)[0, 0]) == 0xAAAAAAAA


def pin_sum_of_terms(o):
    """Residual compensation (Eq. dbf-residual-comp): for l = 1, P = 2 the sum of terms is
    D_a1 S_a1 D_m1 S_b1^T D_b1 + D_a2 S_a2 D_m2 S_b2^T D_b2, written out per entry here; for general
    terms (different k and l) it is the sum of the single-term results."""
    rng = np.random.default_rng(21)
    d_out, d_in = 5, 6
    t1 = rand_layer(rng, d_out, d_in, 4, 1)
    t2 = rand_layer(rng, d_out, d_in, 3, 1)
    W = np.zeros((d_out, d_in))
    for (S_A, S_B, U_A, V_A, U_B, V_B) in (t1, t2):
        a, m, b = U_A[:, 0], V_A[:, 0] * U_B[:, 0], V_B[:, 0]
        for n in range(d_out):
            for i in range(d_in):
                W[n, i] += a[n] * sum(S_A[n, j] * m[j] * S_B[j, i] for j in range(S_A.shape[1])) * b[i]
    assert real.rel_frobenius(o.reconstruct_sum([t1, t2]), W) < 1e-13
    X = rng.standard_normal((d_in, 2))
    assert real.rel_frobenius(o.forward_sum([t1, t2], X), W @ X) < 1e-13
    t3 = rand_layer(rng, d_out, d_in, 7, 3)                   # a third term of another rank
    ref = sum(real.forward(*t, X) for t in (t1, t2, t3))
    assert real.rel_frobenius(o.forward_sum([t1, t2, t3], X), ref) < 1e-13
    assert real.rel_frobenius(o.reconstruct_sum([t3]), real.reconstruct(*t3)) == 0.0
    with pytest.raises(ValueError):
        o.reconstruct_sum([t1, rand_layer(rng, d_out + 1, d_in, 2, 1)])


ALL_PINS = [pin_worked_example, pin_sum_of_dbf, pin_l1_is_dbf, pin_all_plus_signs,
            pin_gauge_and_flips, pin_demodulation_and_isometry, pin_linearity_and_duality,
            pin_metric, pin_packing, pin_sum_of_terms]


@pytest.mark.parametrize("pin", ALL_PINS, ids=lambda f: f.__name__)
def test_pin(pin):
    pin(real)


# ---------------------------------------------------------- brute force
def test_brute_force_all_sign_patterns_4x4x2():
    """Every one of the 2^16 sign patterns of a d_out = d_in = 4, k = 2 instance
    (l = 1 and l = 2): numpy oracle == scalar-loop C twin == an independent
    element-wise evaluation done here with integer sign arithmetic."""
    rng = np.random.default_rng(21)
    d, k = 4, 2
    for l in (1, 2):
        U_A, V_A = rng.standard_normal((d, l)), rng.standard_normal((k, l))
        U_B, V_B = rng.standard_normal((k, l)), rng.standard_normal((d, l))
        x = rng.standard_normal((d, 1))
        E_A = np.einsum("nt,jt->nj", U_A, V_A)
        E_B = np.einsum("js,is->ji", U_B, V_B)
        pats = np.array(list(itertools.product([1, -1], repeat=8)), dtype=np.int8)   # 256 x 8
        SA_all = pats.reshape(256, d, k)
        SB_all = pats.reshape(256, k, d)
        # vectorised independent evaluation: W[a,b,n,i] = sum_j SA[a,n,j] E_A[n,j] SB[b,j,i] E_B[j,i]
        W_all = np.einsum("anj,nj,bji,ji->abni", SA_all.astype(float), E_A, SB_all.astype(float), E_B)
        step = 1
        worst = 0.0
        for a in range(0, 256, step):
            for b in range(0, 256, step):
                W = real.reconstruct(SA_all[a], SB_all[b], U_A, V_A, U_B, V_B)
                worst = max(worst, np.max(np.abs(W - W_all[a, b])))
        assert worst < 1e-13
        # the C twin on a stride of the patterns plus forward agreement
        for a in range(0, 256, 5):
            for b in range(0, 256, 7):
                Wc = loops.reconstruct(SA_all[a], SB_all[b], U_A, V_A, U_B, V_B)
                assert np.max(np.abs(Wc - W_all[a, b])) < 1e-13
                yc = loops.forward(SA_all[a], SB_all[b], U_A, V_A, U_B, V_B, x)
                yo = real.forward(SA_all[a], SB_all[b], U_A, V_A, U_B, V_B, x)
                assert np.max(np.abs(yc - yo)) < 1e-12


def test_loops_twin_matches_numpy_on_random_shapes():
    rng = np.random.default_rng(22)
    for (d_out, d_in, k, l, T) in [(9, 13, 6, 3, 2), (33, 17, 40, 4, 5), (2, 3, 1, 1, 1)]:
        lay = rand_layer(rng, d_out, d_in, k, l)
        X = rng.standard_normal((d_in, T))
        assert real.rel_frobenius(loops.reconstruct(*lay), real.reconstruct(*lay)) < 1e-13
        assert real.rel_frobenius(loops.forward(*lay, X), real.forward(*lay, X)) < 1e-13


# ----------------------------------------------- Theorem 1 / exact projection
def test_fixed_mask_projection_error_is_singular_value_tail():
    """min over F_l(S) of ||U - U_hat||_F^2 = sum_{i>l} sigma_i(S (.) U)^2 (Theorem 1),
    the minimiser lies in F_l(S), and no random member of F_l(S) does better."""
    rng = np.random.default_rng(31)
    N, R = 14, 9
    U = rng.standard_normal((N, R))
    S = rng.choice(np.array([-1, 1], dtype=np.int8), size=(N, R))
    prev = np.inf
    for l in range(1, R + 1):
        P, sv = real.project_fixed_mask(S, U, l)
        err2 = np.sum((U - P) ** 2)
        np.testing.assert_allclose(err2, np.sum(np.linalg.svd(S * U, compute_uv=False)[l:] ** 2),
                                   rtol=1e-10, atol=1e-12)
        assert np.linalg.matrix_rank(S * P, tol=1e-9) <= l
        assert err2 <= prev + 1e-12            # F_1 subset F_l: error can only decrease
        prev = err2
        for _ in range(5):
            cand = real.modulated_factor(S, rng.standard_normal((N, l)), rng.standard_normal((R, l)))
            assert np.sum((U - cand) ** 2) >= err2 - 1e-12
    assert prev < 1e-20                         # l = min(N,R): lossless


def test_msvid_keeps_sign_mask_and_rank():
    """MSVID_l[Z] = sign(Z) (.) TSVD_l(|Z|) with sign(0) = +1 (Eq. msvid-def)."""
    rng = np.random.default_rng(32)
    Z = rng.standard_normal((10, 6))
    Z[0, 0] = 0.0
    for l in (1, 2, 6):
        S, U, V = real.msvid(Z, l)
        assert S[0, 0] == 1
        np.testing.assert_array_equal(S, np.where(Z >= 0, 1, -1))
        E = U @ V.T
        assert np.linalg.matrix_rank(E, tol=1e-9) <= l
        tail = np.linalg.svd(np.abs(Z), compute_uv=False)[l:]
        np.testing.assert_allclose(np.sum((np.abs(Z) - E) ** 2), np.sum(tail ** 2), rtol=1e-9, atol=1e-12)
    S, U, V = real.msvid(Z, 6)
    np.testing.assert_allclose(real.modulated_factor(S, U, V), Z, atol=1e-10)   # full rank: exact


# ------------------------------------------------------- storage accounting
def test_bits_per_weight_and_inner_rank():
    # DBF (l = 1) storage: k (N + M) sign bits + 16 (N + M + 2k) bits of vectors, hand-evaluated
    assert real.bits_per_weight(4, 4, 2, 1) == (2 * 8 + 16 * (4 + 4 + 2 + 2)) / 16.0
    # the workloads' inner ranks are the largest multiples of 128 within budget
    from paper_2512_24545_b200 import inputs
    assert real.largest_inner_rank(4096, 4096, 16, 1.0) == 1664
    assert real.largest_inner_rank(4096, 4096, 16, 1.5) == 2560
    assert real.largest_inner_rank(11008, 4096, 16, 1.5) == 3968
    for (d_out, d_in, l), (k10, k15) in inputs.PREFILL_K.items():
        assert real.largest_inner_rank(d_out, d_in, l, 1.0) == k10
        assert real.largest_inner_rank(d_out, d_in, l, 1.5) == k15
    for name, d_out, d_in, k in inputs.BLOCK70B:
        assert real.largest_inner_rank(d_out, d_in, 16, 1.0) == k
        assert real.bits_per_weight(d_out, d_in, k, 16) <= 1.0 < real.bits_per_weight(d_out, d_in, k + 128, 16)


# --------------------------------------------------- planted mistakes
def _mutants():
    """Broken copies of the oracle; each must fail at least one pin."""
    def ns(**kw):
        d = {n: getattr(real, n) for n in real.__all__}
        d.update(kw)
        return types.SimpleNamespace(**d)

    def rebuilt(mod_factor=None, env=None):
        env = env or real.envelope

        def mf(S, U, V):
            if mod_factor is not None:
                return mod_factor(S, U, V)
            return np.asarray(S, dtype=float) * env(U, V)

        def rec(S_A, S_B, U_A, V_A, U_B, V_B):
            return mf(S_A, U_A, V_A) @ mf(S_B, U_B, V_B)

        def rows(r, S_A, S_B, U_A, V_A, U_B, V_B):
            return rec(S_A, S_B, U_A, V_A, U_B, V_B)[np.asarray(r)]

        def fwd(S_A, S_B, U_A, V_A, U_B, V_B, X):
            return rec(S_A, S_B, U_A, V_A, U_B, V_B) @ np.asarray(X, dtype=float)
        return ns(envelope=env, modulated_factor=mf, reconstruct=rec, reconstruct_rows=rows, forward=fwd)

    m = {}
    m["sign dropped"] = rebuilt(mod_factor=lambda S, U, V: real.envelope(U, V))
    m["last envelope mode dropped"] = rebuilt(
        env=lambda U, V: np.asarray(U, float)[:, :max(1, U.shape[1] - 1)] @ np.asarray(V, float)[:, :max(1, U.shape[1] - 1)].T
        if np.asarray(U).shape[1] > 1 else np.asarray(U, float) @ np.asarray(V, float).T)
    m["sign negated"] = rebuilt(mod_factor=lambda S, U, V: -np.asarray(S, float) * real.envelope(U, V))

    def rec_swapped(S_A, S_B, U_A, V_A, U_B, V_B):     # V_A and U_B (both k x l) exchanged
        return real.reconstruct(S_A, S_B, U_A, U_B, V_A, V_B)
    m["inner factors swapped"] = ns(reconstruct=rec_swapped,
                                    forward=lambda *a: rec_swapped(*a[:6]) @ np.asarray(a[6], float))

    def fwd_T(S_A, S_B, U_A, V_A, U_B, V_B, X):
        W = real.reconstruct(S_A, S_B, U_A, V_A, U_B, V_B)
        return (W.T if W.shape[0] == W.shape[1] else W) @ np.asarray(X, float)
    m["transposed apply on square layers"] = ns(forward=fwd_T)

    def staged_no_mid(S_A, S_B, U_A, V_A, U_B, V_B, X):
        Y, Z = real.forward_staged(S_A, S_B, U_A, V_A, U_B, np.abs(V_B), X)
        return Y, Z
    m["staged order with |V_B|"] = ns(forward_staged=staged_no_mid)
    m["rows off by one"] = ns(reconstruct_rows=lambda r, *a: real.reconstruct(*a)[(np.asarray(r) + 1) % a[0].shape[0]])
    m["metric normalised by the wrong operand"] = ns(rel_frobenius=lambda A, B: real.rel_frobenius(B, A))
    m["pack polarity"] = ns(pack_signs=lambda S: real.pack_signs(-np.asarray(S)),
                            unpack_signs=lambda W, c: -real.unpack_signs(W, c))

    def pack_msb(S):
        S = np.asarray(S)
        pad = (-S.shape[1]) % 32
        bits = np.pad((S == -1).astype(np.uint8), ((0, 0), (0, pad)))
        return np.packbits(bits, axis=1, bitorder="big").view(">u4").astype(np.uint32)
    m["pack MSB first"] = ns(pack_signs=pack_msb)
    m["sum keeps only the first term"] = ns(reconstruct_sum=lambda ts: real.reconstruct(*list(ts)[0]),
                                            forward_sum=lambda ts, X: real.forward(*list(ts)[0], X))
    m["second term subtracted"] = ns(
        reconstruct_sum=lambda ts: real.reconstruct(*list(ts)[0]) - sum(real.reconstruct(*t) for t in list(ts)[1:]),
        forward_sum=lambda ts, X: real.forward_sum(ts, X))
    return m


@pytest.mark.parametrize("name", sorted(_mutants().keys()))
def test_planted_mistakes_are_caught(name):
    mutant = _mutants()[name]
    caught = []
    for pin in ALL_PINS:
        try:
            pin(mutant)
        except (AssertionError, ValueError, IndexError):
            caught.append(pin.__name__)
    assert caught, f"no pin notices the planted mistake: {name}"
