"""ctypes binding of libmdbf.so — same names as include/mdbf.h, argument
marshalling only.  Every computation runs in the CUDA library; there is no
fallback: if the library has not been built or no sm_100 device is present the
calls raise.

Device buffers are passed as raw addresses (e.g. torch.Tensor.data_ptr());
host buffers as numpy arrays.  Streams are raw cudaStream_t integers
(torch.cuda.current_stream().cuda_stream) or 0.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmdbf.so")

F32, F16, BF16 = 0, 1, 2
KERNEL_AUTO, KERNEL_ALU, KERNEL_PREFILL, KERNEL_TMEM, KERNEL_MAT, KERNEL_I8 = 0, 1, 3, 4, 5, 6
OK = 0
ERR_INVALID_ARG, ERR_SHAPE, ERR_DTYPE, ERR_ALLOC, ERR_CUDA, ERR_ARCH, ERR_TIMEOUT, ERR_VALUE, ERR_BOUNDS = (
    -1, -2, -3, -4, -5, -6, -7, -8, -9)
DTYPES = {"f32": F32, "f16": F16, "bf16": BF16}

EXPORTS = (
    "mdbf_pack_signs", "mdbf_unpack_signs", "mdbf_pack", "mdbf_get_packed", "mdbf_get_envelope",
    "mdbf_get_desc", "mdbf_set_kernel", "mdbf_linear_forward", "mdbf_linear_forward_host", "mdbf_linear_forward_host_async", "mdbf_prepare_host_staging",
    "mdbf_linear_forward_static", "mdbf_linear_forward_sum", "mdbf_linear_forward_siblings", "mdbf_linear_forward_group",
    "mdbf_get_intermediate", "mdbf_reconstruct", "mdbf_msvid", "mdbf_msvid_workspace_bytes", "mdbf_project_fixed_mask", "mdbf_admm_factor_update", "mdbf_admm_workspace_bytes", "mdbf_poll_status", "mdbf_selftest_wait_timeout", "mdbf_debug_fail_alloc",
    "mdbf_last_launch_count",
    "mdbf_last_kernel",
    "mdbf_destroy", "mdbf_last_error", "mdbf_version",
)


class MdbfError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"libmdbf status {status}: {message}")
        self.status = status


class Desc(ctypes.Structure):
    _fields_ = [("d_out", ctypes.c_int32), ("d_in", ctypes.c_int32), ("k", ctypes.c_int32),
                ("l", ctypes.c_int32), ("env_dtype", ctypes.c_int32), ("max_T", ctypes.c_int32)]


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """Load libmdbf.so (built by paper_2512_24545_b200.build); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2512_24545_b200.build` "
            "(there is no CPU fallback)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    L.mdbf_pack_signs.argtypes = [vp, i64, i64, vp, ctypes.c_int, vp]
    L.mdbf_unpack_signs.argtypes = [vp, i64, i64, vp, ctypes.c_int, vp]
    L.mdbf_pack.argtypes = [ctypes.POINTER(Desc), vp, vp, vp, vp, vp, vp, ctypes.c_int, vp,
                            ctypes.POINTER(vp)]
    L.mdbf_get_packed.argtypes = [vp, ctypes.c_int, vp, ctypes.c_int, vp]
    L.mdbf_get_envelope.argtypes = [vp, ctypes.c_int, vp, ctypes.c_int, vp]
    L.mdbf_get_desc.argtypes = [vp, ctypes.POINTER(Desc)]
    L.mdbf_set_kernel.argtypes = [vp, i32]
    L.mdbf_linear_forward.argtypes = [vp, vp, vp, i32, i32, vp]
    L.mdbf_linear_forward_host.argtypes = [vp, vp, vp, i32, i32, vp]
    L.mdbf_linear_forward_host_async.argtypes = [vp, vp, vp, i32, i32, vp]
    L.mdbf_prepare_host_staging.argtypes = [vp]
    L.mdbf_linear_forward_static.argtypes = [ctypes.POINTER(Desc), vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, vp]
    L.mdbf_linear_forward_sum.argtypes = [vp, i32, vp, vp, vp, i32, i32, vp]
    L.mdbf_linear_forward_siblings.argtypes = [vp, i32, vp, vp, i32, i32, vp]
    L.mdbf_linear_forward_group.argtypes = [vp, i32, vp, vp, i32, i32, vp]
    L.mdbf_get_intermediate.argtypes = [vp, vp, i32, ctypes.c_int, vp]
    L.mdbf_reconstruct.argtypes = [vp, vp, vp]
    L.mdbf_msvid.argtypes = [vp, i64, i64, i32, i32, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    L.mdbf_project_fixed_mask.argtypes = [vp, vp, i64, i64, i32, i32, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    L.mdbf_msvid_workspace_bytes.argtypes = [i64, i64, i32, ctypes.POINTER(ctypes.c_size_t)]
    L.mdbf_admm_workspace_bytes.argtypes = [i64, i64, i64, i32, ctypes.POINTER(ctypes.c_size_t)]
    L.mdbf_admm_factor_update.argtypes = [vp, i64, i64, i32, vp, i64, vp, vp, ctypes.c_float, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp,
                                          ctypes.c_size_t, vp]
    L.mdbf_poll_status.argtypes = [vp, ctypes.POINTER(i32)]
    L.mdbf_selftest_wait_timeout.argtypes = [vp, vp]
    L.mdbf_debug_fail_alloc.argtypes = [i32]
    L.mdbf_last_launch_count.argtypes = [vp, ctypes.POINTER(i32)]
    L.mdbf_last_kernel.argtypes = [vp, ctypes.POINTER(i32)]
    L.mdbf_destroy.argtypes = [vp]
    for name in EXPORTS:
        getattr(L, name).restype = i32
    L.mdbf_last_error.restype = ctypes.c_char_p
    L.mdbf_last_error.argtypes = []
    L.mdbf_version.restype = ctypes.c_char_p
    L.mdbf_version.argtypes = []
    L.mdbf_debug_fail_alloc.restype = None
    _lib = L
    return L


def last_error() -> str:
    return lib().mdbf_last_error().decode()


def version() -> str:
    return lib().mdbf_version().decode()


def _check(status: int) -> None:
    if status != OK:
        raise MdbfError(status, last_error())


def _addr(buf) -> int:
    """Raw address of a numpy array (host) or an int (device pointer)."""
    if isinstance(buf, np.ndarray):
        if not buf.flags["C_CONTIGUOUS"]:
            raise ValueError("host buffers must be C-contiguous")
        return buf.ctypes.data
    if buf is None:
        return 0
    return int(buf)


def mdbf_pack_signs(s, rows: int, cols: int, out, on_device: bool, stream: int = 0) -> None:
    _check(lib().mdbf_pack_signs(_addr(s), rows, cols, _addr(out), int(on_device), stream))


def mdbf_unpack_signs(p, rows: int, cols: int, out, on_device: bool, stream: int = 0) -> None:
    _check(lib().mdbf_unpack_signs(_addr(p), rows, cols, _addr(out), int(on_device), stream))


def mdbf_pack(d_out: int, d_in: int, k: int, l: int, env_dtype: int, max_T: int,
              S_A, S_B, U_A, V_A, U_B, V_B, inputs_on_device: bool = False, stream: int = 0) -> int:
    """Returns the handle (an integer address)."""
    desc = Desc(d_out, d_in, k, l, env_dtype, max_T)
    h = ctypes.c_void_p()
    _check(lib().mdbf_pack(ctypes.byref(desc), _addr(S_A), _addr(S_B), _addr(U_A), _addr(V_A),
                           _addr(U_B), _addr(V_B), int(inputs_on_device), stream, ctypes.byref(h)))
    return h.value


def mdbf_get_packed(h: int, which: int, out, out_on_device: bool = False, stream: int = 0) -> None:
    _check(lib().mdbf_get_packed(h, which, _addr(out), int(out_on_device), stream))


def mdbf_get_envelope(h: int, which: int, out, out_on_device: bool = False, stream: int = 0) -> None:
    _check(lib().mdbf_get_envelope(h, which, _addr(out), int(out_on_device), stream))


def mdbf_get_desc(h: int) -> Desc:
    d = Desc()
    _check(lib().mdbf_get_desc(h, ctypes.byref(d)))
    return d


def mdbf_set_kernel(h: int, kernel: int) -> None:
    _check(lib().mdbf_set_kernel(h, kernel))


def mdbf_linear_forward(h: int, x, y, T: int, act_dtype: int, stream: int = 0) -> None:
    _check(lib().mdbf_linear_forward(h, _addr(x), _addr(y), T, act_dtype, stream))


def mdbf_linear_forward_sum(handles, x, y, acc, T: int, act_dtype: int, stream: int = 0) -> None:
    """y = sum_p W_hat^(p) x over the given layer handles; acc is a device float32 T x d_out scratch."""
    arr = (ctypes.c_void_p * len(handles))(*handles)
    _check(lib().mdbf_linear_forward_sum(ctypes.cast(arr, ctypes.c_void_p), len(handles), _addr(x), _addr(y), _addr(acc),
                                         T, act_dtype, stream))


def mdbf_linear_forward_siblings(handles, x, ys, T: int, act_dtype: int, stream: int = 0) -> None:
    """ys[i] = W_hat_i x for layers that share the input x (q/k/v, gate/up); ys are device addresses."""
    hs = (ctypes.c_void_p * len(handles))(*handles)
    outs = (ctypes.c_void_p * len(ys))(*[_addr(y) for y in ys])
    _check(lib().mdbf_linear_forward_siblings(ctypes.cast(hs, ctypes.c_void_p), len(handles), _addr(x),
                                              ctypes.cast(outs, ctypes.c_void_p), T, act_dtype, stream))


def mdbf_linear_forward_group(handles, xs, ys, T: int, act_dtype: int, stream: int = 0) -> None:
    """ys[i] = W_hat_i xs[i] for independent layers (own inputs); xs, ys are device addresses."""
    hs = (ctypes.c_void_p * len(handles))(*handles)
    ins = (ctypes.c_void_p * len(xs))(*[_addr(x) for x in xs])
    outs = (ctypes.c_void_p * len(ys))(*[_addr(y) for y in ys])
    _check(lib().mdbf_linear_forward_group(ctypes.cast(hs, ctypes.c_void_p), len(handles), ctypes.cast(ins, ctypes.c_void_p),
                                           ctypes.cast(outs, ctypes.c_void_p), T, act_dtype, stream))


def mdbf_prepare_host_staging(h: int) -> None:
    """Allocate the handle's device staging buffers for mdbf_linear_forward_host (once per handle)."""
    _check(lib().mdbf_prepare_host_staging(h))


def mdbf_linear_forward_host(h: int, x_host, y_host, T: int, act_dtype: int, stream: int = 0) -> None:
    _check(lib().mdbf_linear_forward_host(h, _addr(x_host), _addr(y_host), T, act_dtype, stream))


def mdbf_linear_forward_host_async(h: int, x_host, y_host, T: int, act_dtype: int, stream: int = 0) -> None:
    """Host buffers, no synchronisation: y_host is valid once the caller has synchronised `stream`."""
    _check(lib().mdbf_linear_forward_host_async(h, _addr(x_host), _addr(y_host), T, act_dtype, stream))


STATIC_MAX_KT = 262144


def mdbf_linear_forward_static(d_out: int, d_in: int, k: int, l: int, env_dtype: int, wA, wB, U_A, V_A, U_B, V_B,
                               x, y, T: int, act_dtype: int, stream: int = 0) -> None:
    """Forward for callers that may not allocate device memory: no handle, every buffer (packed
    words, envelopes stored in env_dtype, x, y) is a device address the caller owns; the k x T
    intermediate sits in a fixed array inside the library (k * T <= STATIC_MAX_KT).  Calls on one
    device share that array and must not overlap; make the first call outside stream capture."""
    desc = Desc(d_out, d_in, k, l, env_dtype, T)
    _check(lib().mdbf_linear_forward_static(ctypes.byref(desc), _addr(wA), _addr(wB), _addr(U_A), _addr(V_A),
                                            _addr(U_B), _addr(V_B), _addr(x), _addr(y), T, act_dtype, stream))


def mdbf_get_intermediate(h: int, z, T: int, out_on_device: bool = False, stream: int = 0) -> None:
    _check(lib().mdbf_get_intermediate(h, _addr(z), T, int(out_on_device), stream))


def mdbf_reconstruct(h: int, W, stream: int = 0) -> None:
    _check(lib().mdbf_reconstruct(h, _addr(W), stream))


def mdbf_poll_status(h: int) -> int:
    v = ctypes.c_int32()
    _check(lib().mdbf_poll_status(h, ctypes.byref(v)))
    return v.value


def mdbf_msvid_workspace_bytes(rows: int, cols: int, l: int) -> int:
    v = ctypes.c_size_t()
    _check(lib().mdbf_msvid_workspace_bytes(rows, cols, l, ctypes.byref(v)))
    return v.value


def mdbf_msvid(Z, rows: int, cols: int, l: int, n_iter: int, Q0, S_packed, U, V, sigma, workspace, workspace_bytes: int,
               stream: int = 0) -> None:
    """MSVID_l[Z] = sign(Z) (.) TSVD_l(|Z|) of a device matrix (all arguments device addresses): packed sign mask,
    balanced envelope factors and singular values; asynchronous, the caller owns the workspace.  See include/mdbf.h."""
    _check(lib().mdbf_msvid(_addr(Z), rows, cols, l, n_iter, _addr(Q0), _addr(S_packed), _addr(U), _addr(V), _addr(sigma),
                            _addr(workspace), workspace_bytes, stream))


def mdbf_project_fixed_mask(Z, S_packed, rows: int, cols: int, l: int, n_iter: int, Q0, U, V, sigma, workspace, workspace_bytes: int,
                            stream: int = 0) -> None:
    """S (.) TSVD_l(S (.) Z) for a given packed mask S (Theorem 1's minimiser): balanced factors of the envelope and its
    singular values; device addresses throughout, asynchronous.  See include/mdbf.h."""
    _check(lib().mdbf_project_fixed_mask(_addr(Z), _addr(S_packed), rows, cols, l, n_iter, _addr(Q0), _addr(U), _addr(V), _addr(sigma),
                                         _addr(workspace), workspace_bytes, stream))


def mdbf_admm_workspace_bytes(n: int, m: int, r: int, l: int) -> int:
    v = ctypes.c_size_t()
    _check(lib().mdbf_admm_workspace_bytes(n, m, r, l, ctypes.byref(v)))
    return v.value


def mdbf_admm_factor_update(W, w_rows: int, w_cols: int, transpose_w: bool, V, r: int, U, Lambda, rho: float, l: int, n_inner: int,
                            n_iter: int, Q0, S_packed, Ul, Vl, sigma, U_tilde, workspace, workspace_bytes: int, stream: int = 0) -> None:
    """n_inner ADMM inner iterations on the factor U (N x R dense, updated in place with its dual Lambda) for
    ||op(W) - U V^T||_F^2 with V fixed, the prox step being MSVID_l; device addresses throughout (U_tilde may be None),
    asynchronous.  See include/mdbf.h."""
    _check(lib().mdbf_admm_factor_update(_addr(W), w_rows, w_cols, int(bool(transpose_w)), _addr(V), r, _addr(U), _addr(Lambda),
                                         float(rho), l, n_inner, n_iter, _addr(Q0), _addr(S_packed), _addr(Ul), _addr(Vl), _addr(sigma),
                                         _addr(U_tilde) if U_tilde is not None else None, _addr(workspace), workspace_bytes, stream))


def mdbf_debug_fail_alloc(nth: int) -> None:
    """Test hook: the nth device allocation this thread makes inside the library from now on fails (nth <= 0: cancel)."""
    lib().mdbf_debug_fail_alloc(nth)


def mdbf_selftest_wait_timeout(h: int, stream: int = 0) -> None:
    """Launch the bounded-wait self-test: about a second later the handle's status word reads ERR_TIMEOUT."""
    _check(lib().mdbf_selftest_wait_timeout(h, stream))


def mdbf_last_launch_count(h: int) -> int:
    v = ctypes.c_int32()
    _check(lib().mdbf_last_launch_count(h, ctypes.byref(v)))
    return v.value


def mdbf_last_kernel(h: int) -> int:
    """The KERNEL_* constant of the kernel the last forward on this handle ran (0 before the first)."""
    v = ctypes.c_int32()
    _check(lib().mdbf_last_kernel(h, ctypes.byref(v)))
    return v.value


def mdbf_destroy(h: int) -> None:
    _check(lib().mdbf_destroy(h))
