"""CPU oracle for the MDBF quantized linear forward  y = W_hat x.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain, fp64 statement of
what the CUDA library must compute.  Only tests/, __graft_entry__.smoke() and
the cpu_baseline / --impl reference legs of bench.py may import it; the
product path never does.  It shares no code with the CUDA path and imports
nothing from the package.

Notation (paper, Section "Notation" and Eq. me-dbf-basis), column convention:

    W_hat = U_hat V_hat^T                       (d_out x d_in)
    U_hat = S_A (.) (U_A V_A^T)                 S_A in {+-1}^{d_out x k}
    V_hat^T = S_B (.) (U_B V_B^T)               S_B in {+-1}^{k x d_in}

with the paper's names  S_a = S_A, A = U_A, Q = V_A, S_b = S_B^T, G = U_B,
B = V_B, R = k, N = d_out, M = d_in.  The paper writes the inference with
row vectors (Y = X W_hat, paragraph "Inference"); the format is symmetric
under transposition, so this library uses y = W_hat x with x of shape
(d_in, T).

Every function takes plain numpy arrays of *stored* values (signs as +-1
integers, envelopes and activations already rounded to their storage type)
and computes in float64.

Pins (tests/test_oracle_pins.py): sum-of-DBF expansion (Eq. me-dbf-sum), the
l = 1 DBF product (Eq. dbf-basis), all-(+1) signs, brute force over every sign
pattern of a 4x4x2 instance against the scalar-loop C twin, gauge flips,
demodulation rank and isometry (Eq. me-dbf-envelope-rank, Lemma sign-mask
isometry), a hand-worked example (tests/golden/), the bit-packing definition
against numpy.packbits, the exact-projection error against the singular-value
tail (Theorem 1); the sum of terms against the two-term product of Eq. dbf-residual-comp written
out per entry and against the sum of single-term forwards.  The ADMM factor update (tests/test_oracle_admm.py):
a scalar instance worked by hand, the stationarity and minimality of its least-squares step, the limit of a large
penalty, the fixed point at an exactly representable factor, the envelope rank of its result.  No function here is
"parity unpinned".
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "envelope", "modulated_factor", "reconstruct", "reconstruct_rows", "forward",
    "forward_staged", "reconstruct_sum", "forward_sum", "rel_frobenius", "pack_signs", "unpack_signs",
    "bits_per_weight", "largest_inner_rank", "project_fixed_mask", "msvid", "admm_factor_update",
]


def _f64(a):
    return np.asarray(a, dtype=np.float64)


def _check_signs(S):
    S = np.asarray(S)
    if not np.all((S == 1) | (S == -1)):
        raise ValueError("sign matrix entries must be +1 or -1")
    return S.astype(np.float64)


def envelope(U, V):
    """Demodulated envelope E = U V^T of rank <= l (Eq. me-dbf-envelope-rank)."""
    U, V = _f64(U), _f64(V)
    if U.ndim != 2 or V.ndim != 2 or U.shape[1] != V.shape[1]:
        raise ValueError("envelope factors must be (p x l) and (q x l)")
    return U @ V.T


def modulated_factor(S, U, V):
    """S (.) (U V^T): a member of the class F_l(S) (Definition of F_l, Eq. me-dbf-basis)."""
    S = _check_signs(S)
    E = envelope(U, V)
    if S.shape != E.shape:
        raise ValueError(f"sign matrix {S.shape} does not match envelope {E.shape}")
    return S * E


def reconstruct(S_A, S_B, U_A, V_A, U_B, V_B):
    """Dense W_hat = (S_A (.) U_A V_A^T)(S_B (.) U_B V_B^T)  (Eq. me-dbf-basis).

    Shapes: S_A d_out x k, S_B k x d_in, U_A d_out x l, V_A k x l, U_B k x l,
    V_B d_in x l.  Returns d_out x d_in float64.
    """
    U_hat = modulated_factor(S_A, U_A, V_A)          # d_out x k
    V_hat_T = modulated_factor(S_B, U_B, V_B)        # k x d_in
    if U_hat.shape[1] != V_hat_T.shape[0]:
        raise ValueError("inner rank k of the two factors differs")
    return U_hat @ V_hat_T


def reconstruct_rows(rows, S_A, S_B, U_A, V_A, U_B, V_B):
    """Rows `rows` of W_hat: the definition restricted to a row subset.

    Used for sampled parity at sizes where the dense d_out x d_in product is
    too slow: W_hat[rows, :] = U_hat[rows, :] V_hat^T.
    """
    rows = np.asarray(rows, dtype=np.int64)
    U_hat_rows = modulated_factor(np.asarray(S_A)[rows], _f64(U_A)[rows], V_A)
    V_hat_T = modulated_factor(S_B, U_B, V_B)
    return U_hat_rows @ V_hat_T


def forward(S_A, S_B, U_A, V_A, U_B, V_B, X):
    """Y = W_hat X with W_hat materialised densely; X is d_in x T (or d_in,)."""
    X = _f64(X)
    W = reconstruct(S_A, S_B, U_A, V_A, U_B, V_B)
    if X.shape[0] != W.shape[1]:
        raise ValueError("activation rows must equal d_in")
    return W @ X


def forward_staged(S_A, S_B, U_A, V_A, U_B, V_B, X):
    """The interleaved evaluation order (Eq. DBF-inference-form with the
    expansion of Eq. me-dbf-expand), transposed to the column convention:

        Z = sum_s D_{g^(s)} S_B D_{b^(s)} X          (k x T)
        Y = sum_t D_{a^(t)} S_A D_{q^(t)} Z          (d_out x T)

    Returns (Y, Z).  Z is the k-length intermediate the kernels keep on chip;
    tests use it to localise a disagreement to one stage.
    """
    X = _f64(X)
    S_A = _check_signs(S_A)
    S_B = _check_signs(S_B)
    U_A, V_A, U_B, V_B = _f64(U_A), _f64(V_A), _f64(U_B), _f64(V_B)
    l = U_A.shape[1]
    vec = X.ndim == 1
    if vec:
        X = X[:, None]
    Z = np.zeros((S_B.shape[0], X.shape[1]))
    for s in range(l):
        Z += U_B[:, s:s + 1] * (S_B @ (V_B[:, s:s + 1] * X))
    Y = np.zeros((S_A.shape[0], X.shape[1]))
    for t in range(l):
        Y += U_A[:, t:t + 1] * (S_A @ (V_A[:, t:t + 1] * Z))
    if vec:
        return Y[:, 0], Z[:, 0]
    return Y, Z


def reconstruct_sum(terms):
    """Dense sum of P layers, W_hat = sum_p W_hat^(p): the residual-compensation form
    (Eq. dbf-residual-comp writes it for two DBF terms, i.e. l = 1, P = 2; the paper's (l, P) sweep
    uses MDBF terms).  `terms` is a sequence of (S_A, S_B, U_A, V_A, U_B, V_B) tuples of equal
    d_out and d_in; inner rank and envelope rank may differ between terms."""
    terms = list(terms)
    if not terms:
        raise ValueError("at least one term")
    W = reconstruct(*terms[0])
    for t in terms[1:]:
        Wp = reconstruct(*t)
        if Wp.shape != W.shape:
            raise ValueError("terms must share d_out and d_in")
        W = W + Wp
    return W


def forward_sum(terms, X):
    """Y = (sum_p W_hat^(p)) X with the sum materialised densely first."""
    X = _f64(X)
    W = reconstruct_sum(terms)
    if X.shape[0] != W.shape[1]:
        raise ValueError("activation rows must equal d_in")
    return W @ X


def rel_frobenius(A, B):
    """||A - B||_F / ||B||_F, the paper's reconstruction-error metric
    (Fig. 1 caption and the reconstruction-error paragraph), B the reference."""
    A, B = _f64(A), _f64(B)
    if A.shape != B.shape:
        raise ValueError("shape mismatch")
    den = np.sqrt(np.sum(B * B))
    num = np.sqrt(np.sum((A - B) ** 2))
    if den == 0.0:
        return 0.0 if num == 0.0 else np.inf
    return float(num / den)


# --------------------------------------------------------------------------
# Bit packing.  The paper only says the sign matrices are stored bit-packed
# (paragraph "Inference", effective bits-per-weight); the layout is this
# library's: 32 signs per uint32 along the reduction (column) dimension,
# column c of a row lives in word c // 32 at bit c % 32 (bit 0 = least
# significant), bit set <=> sign is -1 (so the bit equals the IEEE sign bit of
# the +-1 value).  Columns beyond `cols` in the last word are 0 (= +1).
# --------------------------------------------------------------------------
def pack_signs(S):
    S = np.asarray(S)
    if S.ndim != 2:
        raise ValueError("sign matrix must be 2-D")
    if not np.all((S == 1) | (S == -1)):
        raise ValueError("sign matrix entries must be +1 or -1")
    rows, cols = S.shape
    nwords = (cols + 31) // 32
    out = np.zeros((rows, nwords), dtype=np.uint32)
    for c in range(cols):
        neg = (S[:, c] == -1).astype(np.uint32)
        out[:, c // 32] |= neg << np.uint32(c % 32)
    return out


def unpack_signs(words, cols):
    words = np.asarray(words, dtype=np.uint32)
    if words.ndim != 2:
        raise ValueError("packed words must be 2-D (rows x ceil(cols/32))")
    rows, nwords = words.shape
    if nwords != (cols + 31) // 32:
        raise ValueError("word count does not match cols")
    S = np.empty((rows, cols), dtype=np.int8)
    for c in range(cols):
        bit = (words[:, c // 32] >> np.uint32(c % 32)) & np.uint32(1)
        S[:, c] = np.where(bit == 1, -1, 1)
    return S


# --------------------------------------------------------------------------
# Storage accounting (paragraph "Inference": bits-per-weight is the storage of
# the bit-packed sign bases plus the real-valued factors over the N*M entries;
# Section "Setting": the largest inner rank that meets the budget).
# --------------------------------------------------------------------------
def bits_per_weight(d_out, d_in, k, l, env_bits=16):
    sign_bits = k * (d_in + d_out)
    env_values = l * (d_out + k) + l * (k + d_in)      # U_A, V_A, U_B, V_B
    return (sign_bits + env_bits * env_values) / float(d_out * d_in)


def largest_inner_rank(d_out, d_in, l, bpw, env_bits=16, multiple=128):
    """Largest k (a multiple of `multiple`) with bits_per_weight <= bpw."""
    k = 0
    while bits_per_weight(d_out, d_in, k + multiple, l, env_bits) <= bpw:
        k += multiple
    return k


# --------------------------------------------------------------------------
# Fixed-mask projection and the MSVID operator (Theorem 1 / Proposition
# "Exact projection", Eq. msvid-def).  Not on the forward path; they pin the
# format (a projected factor must be representable with rank-l envelopes) and
# are the first step of the quantizer that is scheduled next.
# --------------------------------------------------------------------------
def _tsvd(E, l):
    Uu, s, Vt = np.linalg.svd(E, full_matrices=False)
    return (Uu[:, :l] * s[:l]) @ Vt[:l], s


def project_fixed_mask(S, Z, l):
    """Pi_{F_l(S)}(Z) = S (.) TSVD_l(S (.) Z); returns (projection, singular values of S(.)Z)."""
    S = _check_signs(S)
    Z = _f64(Z)
    E_l, sv = _tsvd(S * Z, l)
    return S * E_l, sv


def msvid(Z, l):
    """MSVID_l[Z] = sign(Z) (.) TSVD_l(|Z|), sign(0) = +1 (Eq. msvid-def, Notation).

    Returns (S, U, V) with S = sign(Z) as int8 and U (p x l), V (q x l) balanced
    factors of the truncated envelope, TSVD_l(|Z|) = U V^T.
    """
    Z = _f64(Z)
    S = np.where(Z >= 0.0, 1, -1).astype(np.int8)
    Uu, s, Vt = np.linalg.svd(np.abs(Z), full_matrices=False)
    r = np.sqrt(s[:l])
    return S, Uu[:, :l] * r, Vt[:l].T * r


# --------------------------------------------------------------------------
# ADMM refinement of one factor with the other held fixed (Section "ADMM
# Refinement", Eq. admm-U-tilde, Eq. admm-U-prox, Eq. admm-U-dual).  The update
# of the other factor is the same function on the transposed problem.
# --------------------------------------------------------------------------
def admm_factor_update(W, V, U, Lam, rho, l, n_inner=1):
    """n_inner ADMM inner iterations on U (N x R, dense values of the factor) for min ||W - U V^T||_F^2 with V (M x R)
    fixed, auxiliary variable U_tilde and scaled dual variable Lam (N x R):

        U_tilde = (W V + rho (U - Lam)) (V^T V + rho I)^-1        Eq. admm-U-tilde
        U       = MSVID_l[U_tilde + Lam]                          Eq. admm-U-prox
        Lam     = Lam + U_tilde - U                               Eq. admm-U-dual

    Returns (U, Lam, U_tildes, masks): the new U and Lam, and per inner iteration the least-squares iterate and the sign
    mask MSVID chose.
    """
    W, V, U, Lam = _f64(W), _f64(V), _f64(U), _f64(Lam)
    R = V.shape[1]
    if W.shape != (U.shape[0], V.shape[0]) or U.shape[1] != R or Lam.shape != U.shape:
        raise ValueError("shapes do not fit W (N x M), V (M x R), U and Lam (N x R)")
    if not rho > 0:
        raise ValueError("rho must be positive")
    G = V.T @ V + rho * np.eye(R)
    WV = W @ V
    tildes, masks = [], []
    for _ in range(n_inner):
        U_tilde = np.linalg.solve(G, (WV + rho * (U - Lam)).T).T          # G is symmetric
        S, Ul, Vl = msvid(U_tilde + Lam, l)
        U = S * (Ul @ Vl.T)
        Lam = Lam + U_tilde - U
        tildes.append(U_tilde)
        masks.append(S)
    return U, Lam, tildes, masks
