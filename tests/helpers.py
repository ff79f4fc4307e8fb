"""Shared test plumbing: build a layer on the GPU through the C-ABI binding, run
forwards, and evaluate the oracle on the same stored values."""
from __future__ import annotations

import numpy as np
import torch

from oracle import mdbf_oracle as orc
from paper_2512_24545_b200 import inputs, mdbf as M

TORCH_DT = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}
TOL = {"bf16": 5e-3, "f16": 5e-3, "f32": 1e-5}     # relative Frobenius bounds on y
TOL_RECONSTRUCT = 1e-6


class GpuLayer:
    """A packed layer plus the host copies of what went in."""

    def __init__(self, spec: inputs.LayerSpec, max_T: int, lay=None, inputs_on_device: bool = False):
        self.spec = spec
        self.lay = lay if lay is not None else inputs.make_layer(spec)
        L = self.lay
        args = [np.ascontiguousarray(L[n]) for n in ("S_A", "S_B", "U_A", "V_A", "U_B", "V_B")]
        self._keep = args
        if inputs_on_device:
            dev = [torch.from_numpy(a).cuda() for a in args]
            self._keep = dev
            args = [t.data_ptr() for t in dev]
            torch.cuda.synchronize()
        self.h = M.mdbf_pack(spec.d_out, spec.d_in, spec.k, spec.l, M.DTYPES[spec.env_dtype], max_T,
                             *args, inputs_on_device=inputs_on_device)
        self.max_T = max_T

    def close(self):
        if self.h:
            M.mdbf_destroy(self.h)
            self.h = 0

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # ---- GPU side
    def forward(self, x: np.ndarray, kernel: int = M.KERNEL_AUTO, act_dtype: str | None = None) -> np.ndarray:
        """x: (T, d_in) float32 holding act_dtype-representable values -> y (T, d_out) float32."""
        act = act_dtype or self.spec.act_dtype
        T = x.shape[0]
        xd = torch.from_numpy(np.ascontiguousarray(x)).to(TORCH_DT[act]).cuda()
        yd = torch.full((T, self.spec.d_out), float("nan"), dtype=TORCH_DT[act], device="cuda")
        M.mdbf_set_kernel(self.h, kernel)
        M.mdbf_linear_forward(self.h, xd.data_ptr(), yd.data_ptr(), T, M.DTYPES[act],
                              torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        M.mdbf_set_kernel(self.h, M.KERNEL_AUTO)
        return yd.to(torch.float32).cpu().numpy()

    def intermediate(self, T: int) -> np.ndarray:
        z = np.empty((T, self.spec.k), dtype=np.float32)
        M.mdbf_get_intermediate(self.h, z, T)
        return z

    def reconstruct(self) -> np.ndarray:
        W = torch.empty((self.spec.d_out, self.spec.d_in), dtype=torch.float32, device="cuda")
        M.mdbf_reconstruct(self.h, W.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        return W.cpu().numpy()

    # ---- oracle side (same stored values)
    def oracle_args(self):
        L = self.lay
        return (L["S_A"], L["S_B"], L["U_A"], L["V_A"], L["U_B"], L["V_B"])

    def oracle_forward(self, x: np.ndarray) -> np.ndarray:
        """(T, d_in) -> (T, d_out) float64, dense definition."""
        return orc.forward(*self.oracle_args(), x.T.astype(np.float64)).T

    def oracle_forward_rows(self, x: np.ndarray, rows) -> np.ndarray:
        """Outputs for the sampled rows only: (T, len(rows)) float64."""
        W_rows = orc.reconstruct_rows(rows, *self.oracle_args())
        return (W_rows @ x.T.astype(np.float64)).T


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    return orc.rel_frobenius(got, ref)
