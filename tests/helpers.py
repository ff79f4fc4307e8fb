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


GUARD_BYTES = 4096          # on either side of every output buffer of GpuLayer.forward (a multiple of 16: y stays aligned)
GUARD_PATTERN = 0xA5


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
        # the output sits between two guard regions filled with a byte pattern no kernel writes: a store before the
        # first or past the last element of y shows up here (no memory checker runs on the GPU tests)
        n = T * self.spec.d_out
        esz = torch.empty((), dtype=TORCH_DT[act]).element_size()
        guard = GUARD_BYTES // esz
        raw = torch.empty(guard + n + guard, dtype=TORCH_DT[act], device="cuda")
        raw.view(torch.uint8).fill_(GUARD_PATTERN)
        yd = raw[guard:guard + n].view(T, self.spec.d_out)
        yd.fill_(float("nan"))
        M.mdbf_set_kernel(self.h, kernel)
        try:
            M.mdbf_linear_forward(self.h, xd.data_ptr(), yd.data_ptr(), T, M.DTYPES[act],
                                  torch.cuda.current_stream().cuda_stream)
            torch.cuda.synchronize()
        finally:
            M.mdbf_set_kernel(self.h, M.KERNEL_AUTO)
        lo = raw[:guard].view(torch.uint8)
        hi = raw[guard + n:].view(torch.uint8)
        assert bool((lo == GUARD_PATTERN).all()) and bool((hi == GUARD_PATTERN).all()), "a kernel wrote outside y"
        # the device status word: MDBF_ERR_TIMEOUT after a bounded wait expired and, in the bounds-checked build
        # (MDBF_BOUNDS_CHECK=1), MDBF_ERR_BOUNDS after a kernel computed a store index outside its buffer
        status = M.mdbf_poll_status(self.h)
        assert status == 0, f"device status {status} after a forward"
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


def magnitude_bound(g: "GpuLayer", x: np.ndarray, rows=None) -> np.ndarray:
    """|U_hat| (|V_hat^T| |x|) as a (T, d_out) array (or its columns `rows`): what |y| could be if nothing cancelled.  Every rounding on a
    bf16 path perturbs a y element by at most 2^-8 of this (a relative error of one operand or partial result
    propagates through sums of absolute values), whatever the shape - also where k is too small for errors to
    average out."""
    L = g.lay
    sel = slice(None) if rows is None else rows
    Uh = np.abs(orc.modulated_factor(L["S_A"][sel], L["U_A"][sel], L["V_A"]))     # (rows of) d_out x k
    Vh = np.abs(orc.modulated_factor(L["S_B"], L["U_B"], L["V_B"]))               # k x d_in
    return (Uh @ (Vh @ np.abs(x.T.astype(np.float64)))).T


def check_parity(g: "GpuLayer", x: np.ndarray, got: np.ndarray, ref: np.ndarray | None = None, roundings: int = 4,
                 act: str | None = None, averaging: bool = True) -> float:
    """The three parity assertions of a forward against the oracle; returns the whole-array error.
      1. whole array: relative Frobenius error <= 5e-3 (bf16 activations, fp32 accumulation) / 1e-5 (fp32 path);
      2. every block of 128 output rows on its own: the same bound, so that one wrong tile cannot hide in the norm;
      3. every element: |y - y_ref| <= (roundings + 1) * 2^-8 * |U_hat| (|V_hat^T| |x|) (fp32 path: 1e-5 of it),
         `roundings` = bf16 roundings on the path that produced y.
    averaging=False (layers with a handful of terms per output, where rounding errors cannot average out and the
    Frobenius ratio is no sharper than the per-element bound) keeps assertion 3 only."""
    act = act or g.spec.act_dtype
    tol = TOL[act]
    if ref is None:
        ref = g.oracle_forward(x)
    assert got.shape == ref.shape
    assert np.all(np.isfinite(got))
    bound = magnitude_bound(g, x)
    unit = 1e-5 if act == "f32" else (roundings + 1) * 2.0 ** -8
    excess = np.abs(got - ref) - unit * bound
    worst = np.unravel_index(np.argmax(excess), excess.shape)
    assert excess[worst] <= 1e-30, (f"element {worst}: |y - y_ref| = {abs(got[worst] - ref[worst]):.3e} exceeds "
                                    f"{unit:.2e} * {bound[worst]:.3e}")
    err = rel_err(got, ref)
    if not averaging:
        return err
    assert err <= tol, f"relative Frobenius error {err:.3e} > {tol}"
    ref_rms = np.sqrt(np.mean(ref ** 2))
    for r0 in range(0, ref.shape[1], 128):
        blk = slice(r0, min(r0 + 128, ref.shape[1]))
        if blk.stop - blk.start < 128:                                   # a ragged tail of a few rows is too small a sample for a
            continue                                                     # norm ratio: the per-element bound above covers it
        if np.sqrt(np.mean(ref[:, blk] ** 2)) < 1e-3 * ref_rms:          # a block of (nearly) zero rows has no relative error
            continue
        e = rel_err(got[:, blk], ref[:, blk])
        assert e <= tol, f"rows {r0}..{blk.stop - 1}: relative Frobenius error {e:.3e} > {tol}"
    return err
