"""Layer-wise MDBF quantization of a weight matrix on the GPU (Section "Layer-Wise Optimization"): rank-R truncated SVD,
balanced factors (Eq. mesvid-balanced), Multi-Envelope SVID initialisation (Eq. mesvid-init-compact) and alternating
ADMM refinement of the two factors (Eq. admm-U-tilde, Eq. admm-U-prox, Eq. admm-U-dual).

This module only sequences calls: the truncated SVD of W is a library routine (torch.linalg.svd), every step of the method
itself runs in libmdbf (mdbf_msvid, mdbf_admm_factor_update, mdbf_pack); torch supplies device memory, transposes and
the unpacking of the bit masks into the +-1 arrays mdbf_pack takes.

Names follow the paper: W is N x M, the inner dimension is R, U is N x R and V is M x R with W ~ U V^T.  In the
library's layer format (y = W_hat x, W_hat = (S_A (.) U_A V_A^T)(S_B (.) U_B V_B^T)) U is the first factor and V^T the
second, so d_out = N, d_in = M, k = R.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

from . import inputs, mdbf as M


@dataclass
class QuantizedLayer:
    d_out: int
    d_in: int
    k: int
    l: int
    S_A: torch.Tensor       # d_out x k int8 +-1
    S_B: torch.Tensor       # k x d_in int8 +-1
    U_A: torch.Tensor       # d_out x l fp32
    V_A: torch.Tensor       # k x l
    U_B: torch.Tensor       # k x l
    V_B: torch.Tensor       # d_in x l
    err_svd: float          # ||W - W_R||_F / ||W||_F of the rank-R truncation
    err_init: float         # the same for the MSVID initialisation
    err_final: float        # and after the refinement

    def dense(self) -> torch.Tensor:
        """W_hat as the format defines it (fp64 on the device; for checks)."""
        A = self.S_A.double() * (self.U_A.double() @ self.V_A.double().T)
        B = self.S_B.double() * (self.U_B.double() @ self.V_B.double().T)
        return A @ B

    def pack(self, env_dtype: int = M.F16, max_T: int = 64) -> int:
        """A layer handle for mdbf_linear_forward (the envelopes are rounded to env_dtype by mdbf_pack)."""
        host = [t.cpu().numpy() for t in (self.S_A, self.S_B, self.U_A, self.V_A, self.U_B, self.V_B)]
        return M.mdbf_pack(self.d_out, self.d_in, self.k, self.l, env_dtype, max_T, *host)


def _unpack(S_packed: torch.Tensor, cols: int) -> torch.Tensor:
    """rows x ceil(cols / 32) int32 words (bit set <=> -1) -> rows x cols int8 +-1."""
    j = torch.arange(cols, device=S_packed.device)
    bits = (S_packed[:, (j >> 5)] >> (j & 31)) & 1
    return (1 - 2 * bits).to(torch.int8)


def _msvid(Z: torch.Tensor, l: int, n_iter: int, seed: int):
    rows, cols = Z.shape
    Q0 = torch.from_numpy(inputs.make_start_block(cols, l, seed)).to(Z.device)
    S = torch.zeros((rows, (cols + 31) // 32), dtype=torch.int32, device=Z.device)
    Ul = torch.zeros((rows, l), dtype=torch.float32, device=Z.device)
    Vl = torch.zeros((cols, l), dtype=torch.float32, device=Z.device)
    sg = torch.zeros((l,), dtype=torch.float32, device=Z.device)
    nbytes = M.mdbf_msvid_workspace_bytes(rows, cols, l)
    ws = torch.empty(nbytes, dtype=torch.uint8, device=Z.device)
    M.mdbf_msvid(Z.data_ptr(), rows, cols, l, n_iter, Q0.data_ptr(), S.data_ptr(), Ul.data_ptr(), Vl.data_ptr(), sg.data_ptr(),
                 ws.data_ptr(), nbytes, torch.cuda.current_stream().cuda_stream)
    return _unpack(S, cols), Ul, Vl


def quantize_layer(W: torch.Tensor, R: int, l: int, n_alternations: int = 2, n_inner: int = 3, n_iter: int = 8,
                   rho_scale: float = 3.0, seed: int = 0) -> QuantizedLayer:
    """W: N x M fp32 on a CUDA device.  rho = rho_scale x the mean diagonal entry of the fixed factor's Gram matrix (the paper
    gives no value; at a tenth of that scale the scheme diverges and at the scale itself it is not monotone on every matrix,
    in the oracle as here; at three times the scale it refined monotonically on the matrices tried)."""
    if not (W.is_cuda and W.dtype == torch.float32 and W.dim() == 2 and W.is_contiguous()):
        raise ValueError("W must be a contiguous 2-D fp32 CUDA tensor")
    N, Mc = W.shape
    if not (1 <= l <= min(32, R) and R <= min(N, Mc)):
        raise ValueError("need 1 <= l <= min(32, R) and R <= min(N, M)")
    st = torch.cuda.current_stream().cuda_stream
    Uu, s, Vt = torch.linalg.svd(W.double(), full_matrices=False)                      # library routine, fp64
    root = s[:R].sqrt()
    U0 = (Uu[:, :R] * root).float().contiguous()                                       # Eq. mesvid-balanced
    V0 = (Vt[:R].T * root).float().contiguous()
    wn = float(torch.linalg.norm(W.double()))
    err_svd = float(torch.linalg.norm(W.double() - U0.double() @ V0.double().T)) / wn
    # Eq. mesvid-init-compact
    S_U, Ul_U, Vl_U = _msvid(U0, l, n_iter, seed)
    S_V, Ul_V, Vl_V = _msvid(V0, l, n_iter, seed + 1)
    U = (S_U.float() * (Ul_U @ Vl_U.T)).contiguous()
    V = (S_V.float() * (Ul_V @ Vl_V.T)).contiguous()
    err_init = float(torch.linalg.norm(W.double() - U.double() @ V.double().T)) / wn
    # alternating refinement; each factor keeps its dual variable across the alternations
    Lam_U, Lam_V = torch.zeros_like(U), torch.zeros_like(V)
    ws_bytes = max(M.mdbf_admm_workspace_bytes(N, Mc, R, l), M.mdbf_admm_workspace_bytes(Mc, N, R, l))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=W.device) if n_alternations > 0 else None
    Q0 = torch.from_numpy(inputs.make_start_block(R, l, seed + 2)).to(W.device)
    sg = torch.zeros((l,), dtype=torch.float32, device=W.device)

    def update(transpose, fixed, X, Lam):
        rows = X.shape[0]
        S = torch.zeros((rows, (R + 31) // 32), dtype=torch.int32, device=W.device)
        Xl = torch.zeros((rows, l), dtype=torch.float32, device=W.device)
        Rl = torch.zeros((R, l), dtype=torch.float32, device=W.device)
        rho = rho_scale * float((fixed.double() ** 2).sum()) / R
        M.mdbf_admm_factor_update(W.data_ptr(), N, Mc, transpose, fixed.data_ptr(), R, X.data_ptr(), Lam.data_ptr(), rho, l, n_inner,
                                  n_iter, Q0.data_ptr(), S.data_ptr(), Xl.data_ptr(), Rl.data_ptr(), sg.data_ptr(), None, ws.data_ptr(),
                                  ws_bytes, st)
        return _unpack(S, R), Xl, Rl

    for _ in range(n_alternations):
        S_U, Ul_U, Vl_U = update(False, V, U, Lam_U)
        S_V, Ul_V, Vl_V = update(True, U, V, Lam_V)
    err_final = float(torch.linalg.norm(W.double() - U.double() @ V.double().T)) / wn
    if not bool(torch.isfinite(sg).all()):
        raise RuntimeError("the refinement reported a failed step (non-finite singular values)")
    # the library's layer format: first factor U = S_A (.) (U_A V_A^T); second factor V^T = S_V^T (.) (Vl_V Ul_V^T)
    return QuantizedLayer(N, Mc, R, l, S_U.contiguous(), S_V.T.contiguous(), Ul_U, Vl_U, Vl_V, Ul_V, err_svd, err_init, err_final)
