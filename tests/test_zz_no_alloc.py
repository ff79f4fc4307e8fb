"""mdbf_linear_forward_static: the forward for callers that may not allocate device memory
(a runtime that froze its allocator, a plug-in handed buffers by its host, a real-time loop).
It takes packed words and envelopes the caller already holds on the device and keeps the
k x T intermediate in a fixed array inside the library.  Checked here, through the C ABI,
against the handle-based entry point on two calls in a row (the array is shared between
calls and keeps the previous call's contents).  Collected last on purpose."""
import numpy as np
import pytest
import torch

from paper_2512_24545_b200 import inputs, mdbf as M

TOL = {"f32": 1e-5, "bf16": 5e-3}     # the relative Frobenius bounds the parity tests use


def _rel(a, b):
    a, b = a.astype(np.float64), b.astype(np.float64)
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def _device_layer(spec, lay):
    """What a non-allocating caller would already own: canonical words and stored envelopes."""
    tdt = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}[spec.env_dtype]
    st = torch.cuda.current_stream().cuda_stream
    words = []
    for name, rows, cols in (("S_A", spec.d_out, spec.k), ("S_B", spec.k, spec.d_in)):
        s = torch.from_numpy(np.ascontiguousarray(lay[name])).cuda()
        w = torch.zeros((rows, (cols + 31) // 32), dtype=torch.int32, device="cuda")
        M.mdbf_pack_signs(s.data_ptr(), rows, cols, w.data_ptr(), True, st)
        words.append(w)
    env = [torch.from_numpy(np.ascontiguousarray(lay[n])).to(tdt).cuda() for n in ("U_A", "V_A", "U_B", "V_B")]
    torch.cuda.synchronize()
    return words, env


@pytest.mark.gpu
@pytest.mark.parametrize("case", ["fp32_tiny", "bf16_ragged"])
def test_static_forward_matches_handle_forward_twice(case):
    from paper_2512_24545_b200 import build
    build.build()
    if case == "fp32_tiny":
        spec, T = inputs.tiny(), 8
    else:
        spec, T = inputs.scaled(inputs.qproj(1664), name="ragged", d_out=203, d_in=333, k=97, l=5), 3
    act = spec.act_dtype
    tdt = torch.float32 if act == "f32" else torch.bfloat16
    lay = inputs.make_layer(spec)
    words, env = _device_layer(spec, lay)
    st = torch.cuda.current_stream().cuda_stream
    h = M.mdbf_pack(spec.d_out, spec.d_in, spec.k, spec.l, M.DTYPES[spec.env_dtype], T,
                    *[np.ascontiguousarray(lay[n]) for n in ("S_A", "S_B", "U_A", "V_A", "U_B", "V_B")])
    try:
        M.mdbf_set_kernel(h, M.KERNEL_ALU)
        for call in range(2):                      # second call meets the first call's leftovers
            x = torch.from_numpy(inputs.make_activations(spec, T, seed_offset=call)).to(tdt).cuda()
            y_ref = torch.zeros((T, spec.d_out), dtype=tdt, device="cuda")
            y = torch.full((T, spec.d_out), float("nan"), dtype=tdt, device="cuda")
            M.mdbf_linear_forward(h, x.data_ptr(), y_ref.data_ptr(), T, M.DTYPES[act], st)
            M.mdbf_linear_forward_static(spec.d_out, spec.d_in, spec.k, spec.l, M.DTYPES[spec.env_dtype],
                                         words[0].data_ptr(), words[1].data_ptr(),
                                         *[e.data_ptr() for e in env], x.data_ptr(), y.data_ptr(), T,
                                         M.DTYPES[act], st)
            torch.cuda.synchronize()
            got, ref = y.float().cpu().numpy(), y_ref.float().cpu().numpy()
            assert np.all(np.isfinite(got))
            assert _rel(got, ref) <= TOL[act], f"call {call}"
            # and against the CPU oracle itself, on the values as stored (envelopes rounded to the layer's type)
            from oracle import mdbf_oracle as orc
            stored = [e.float().cpu().numpy().astype(np.float64) for e in env]
            y_orc = orc.forward(lay["S_A"], lay["S_B"], stored[0], stored[1], stored[2], stored[3],
                                x.float().cpu().numpy().T.astype(np.float64)).T
            assert _rel(got, y_orc) <= TOL[act], f"call {call} against the oracle"
    finally:
        M.mdbf_destroy(h)


@pytest.mark.gpu
def test_static_forward_rejects_oversize_and_bad_arguments():
    from paper_2512_24545_b200 import build
    build.build()
    buf = torch.zeros(1024, dtype=torch.float32, device="cuda")
    p = buf.data_ptr()
    k = 4096
    T = M.STATIC_MAX_KT // k + 1                  # one token beyond the built-in scratch
    with pytest.raises(M.MdbfError) as e:
        M.mdbf_linear_forward_static(8, 8, k, 1, M.F16, p, p, p, p, p, p, p, p, T, M.BF16)
    assert e.value.status == M.ERR_SHAPE and "MDBF_STATIC_MAX_KT" in str(e.value)
    with pytest.raises(M.MdbfError) as e:
        M.mdbf_linear_forward_static(8, 8, 8, 1, M.F16, p, p, p, p, p, p, 0, p, 1, M.BF16)
    assert e.value.status == M.ERR_INVALID_ARG
    with pytest.raises(M.MdbfError) as e:
        M.mdbf_linear_forward_static(8, 8, 8, 1, 5, p, p, p, p, p, p, p, p, 1, M.BF16)
    assert e.value.status == M.ERR_DTYPE


def test_static_forward_argument_checks_need_no_gpu():
    from paper_2512_24545_b200 import build
    build.build()
    with pytest.raises(M.MdbfError) as e:
        M.mdbf_linear_forward_static(8, 8, 8, 1, M.F16, 0, 0, 0, 0, 0, 0, 0, 0, 1, M.BF16)
    assert e.value.status == M.ERR_INVALID_ARG
    with pytest.raises(M.MdbfError) as e:
        M.mdbf_linear_forward_static(8, 8, 8, 0, M.F16, 1, 1, 1, 1, 1, 1, 1, 1, 1, M.BF16)
    assert e.value.status == M.ERR_SHAPE
    with pytest.raises(M.MdbfError) as e:
        M.mdbf_linear_forward_static(8, 8, 65536, 1, M.F16, 1, 1, 1, 1, 1, 1, 1, 1, 5, M.BF16)
    assert e.value.status == M.ERR_SHAPE
