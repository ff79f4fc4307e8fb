"""Parity of the CUDA path with the CPU oracle, through the C-ABI binding.

Integer work (packing) is compared bit for bit; y by the relative Frobenius
error ||y - y_oracle||_F / ||y_oracle||_F, bound 5e-3 for bf16 activations
(fp32 accumulation) and 1e-5 for the fp32 path; mdbf_reconstruct by 1e-6.
"""
import numpy as np
import pytest
import torch

from oracle import mdbf_oracle as orc
from paper_2512_24545_b200 import inputs, mdbf as M
from helpers import GpuLayer, TOL, TOL_RECONSTRUCT, check_parity, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2512_24545_b200 import build
    build.build()
    assert torch.cuda.is_available()


def small_spec(d_out=352, d_in=544, k=320, l=16, **kw):
    """A reduced q_proj-like layer: several 32x128 sign tiles in both directions with ragged tails."""
    return inputs.scaled(inputs.qproj(1664), name="small", d_out=d_out, d_in=d_in, k=k, l=l, **kw)


# ------------------------------------------------------------------ packing
@pytest.mark.parametrize("rows,cols", [(1, 1), (5, 33), (32, 128), (33, 129), (100, 1000), (7, 4096)])
def test_device_packer_bit_exact(rows, cols):
    rng = np.random.default_rng(rows * 131 + cols)
    S = rng.choice(np.array([-1, 1], dtype=np.int8), size=(rows, cols))
    Sd = torch.from_numpy(S).cuda()
    nw = (cols + 31) // 32
    out = torch.full((rows, nw), -1, dtype=torch.int32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    M.mdbf_pack_signs(Sd.data_ptr(), rows, cols, out.data_ptr(), True, st)
    torch.cuda.synchronize()
    words = out.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(words, orc.pack_signs(S))
    back = torch.zeros((rows, cols), dtype=torch.int8, device="cuda")
    M.mdbf_unpack_signs(out.data_ptr(), rows, cols, back.data_ptr(), True, st)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(back.cpu().numpy(), S)


@pytest.mark.parametrize("on_device", [False, True])
def test_layer_keeps_canonical_words_and_rounded_envelopes(on_device):
    spec = small_spec(d_out=70, d_in=200, k=97, l=5)
    lay = inputs.make_layer(spec)
    # envelope inputs that are NOT fp16-representable: the library rounds them (RNE)
    rng = np.random.default_rng(3)
    raw = {n: (lay[n] * (1 + 1e-4 * rng.standard_normal(lay[n].shape))).astype(np.float32)
           for n in ("U_A", "V_A", "U_B", "V_B")}
    lay2 = dict(lay, **raw)
    with GpuLayer(spec, 4, lay=lay2, inputs_on_device=on_device) as g:
        for which, name, rows, cols in [(0, "S_A", 70, 97), (1, "S_B", 97, 200)]:
            out = np.zeros((rows, (cols + 31) // 32), dtype=np.uint32)
            M.mdbf_get_packed(g.h, which, out)
            np.testing.assert_array_equal(out, orc.pack_signs(lay[name]))
        for which, name in enumerate(("U_A", "V_A", "U_B", "V_B")):
            got = np.zeros_like(raw[name])
            M.mdbf_get_envelope(g.h, which, got)
            np.testing.assert_array_equal(got, inputs.round_to(raw[name], "f16"))
        d = M.mdbf_get_desc(g.h)
        assert (d.d_out, d.d_in, d.k, d.l, d.max_T) == (70, 200, 97, 5, 4)


# -------------------------------------------------------------- reconstruct
@pytest.mark.parametrize("spec", [inputs.tiny(), small_spec(), small_spec(d_out=65, d_in=130, k=33, l=3),
                                  small_spec(l=1), small_spec(env_dtype="bf16")],
                         ids=["tiny", "small", "ragged", "dbf_l1", "bf16_env"])
def test_reconstruct_matches_oracle(spec):
    with GpuLayer(spec, 1) as g:
        W = g.reconstruct()
        ref = orc.reconstruct(*g.oracle_args())
        assert rel_err(W, ref) <= TOL_RECONSTRUCT


# ------------------------------------------------------------ forward, fp32
@pytest.mark.parametrize("T", [1, 8])
def test_tiny_config_fp32(T):
    spec = inputs.tiny()
    x = inputs.make_activations(spec, T)
    with GpuLayer(spec, 8) as g:
        y = g.forward(x)
        assert M.mdbf_last_launch_count(g.h) == 2
        ref = g.oracle_forward(x)
        check_parity(g, x, y, ref)
        z = g.intermediate(T)
        _, z_ref = orc.forward_staged(*g.oracle_args(), x.T.astype(np.float64))
        assert rel_err(z, z_ref.T) <= TOL["f32"]


@pytest.mark.parametrize("shape", [(33, 65, 17, 3), (1, 1, 1, 1), (64, 32, 128, 7), (300, 100, 50, 20)])
def test_alu_path_ragged_shapes_fp32(shape):
    d_out, d_in, k, l = shape
    spec = inputs.scaled(inputs.tiny(), d_out=d_out, d_in=d_in, k=k, l=l)
    x = inputs.make_activations(spec, 3)
    with GpuLayer(spec, 3) as g:
        check_parity(g, x, g.forward(x), averaging=k >= 8)


# ------------------------------------------------------- forward, few tokens, library's choice of kernel
@pytest.mark.parametrize("T", [1, 2, 3, 4])
@pytest.mark.parametrize("l", [1, 4, 16, 24])
def test_few_tokens_small_shapes(T, l):
    spec = small_spec(l=l)
    x = inputs.make_activations(spec, T)
    with GpuLayer(spec, 4) as g:
        ref = g.oracle_forward(x)
        y = g.forward(x)
        check_parity(g, x, y, ref)
        _, z_ref = orc.forward_staged(*g.oracle_args(), x.T.astype(np.float64))
        assert rel_err(g.intermediate(T), z_ref.T) <= TOL["bf16"]
        y_alu = g.forward(x, kernel=M.KERNEL_ALU)
        check_parity(g, x, y_alu, ref, roundings=1)
        assert rel_err(y, y_alu) <= 2 * TOL["bf16"]


@pytest.mark.parametrize("shape", [(1, 1, 1, 1), (31, 127, 33, 2), (32, 128, 128, 16), (129, 1025, 257, 9),
                                   (1000, 2100, 1300, 16)])
def test_few_tokens_edge_shapes(shape):
    d_out, d_in, k, l = shape
    spec = small_spec(d_out=d_out, d_in=d_in, k=k, l=l)
    x = inputs.make_activations(spec, 2)
    with GpuLayer(spec, 2) as g:
        check_parity(g, x, g.forward(x), averaging=k >= 8)


def test_bf16_envelopes_and_repeat_calls():
    spec = small_spec(env_dtype="bf16")
    x = inputs.make_activations(spec, 1)
    with GpuLayer(spec, 1) as g:
        ref = g.oracle_forward(x)
        y1 = g.forward(x)
        y2 = g.forward(x)
        assert rel_err(y1, ref) <= TOL["bf16"]
        np.testing.assert_array_equal(y1, y2)          # deterministic: no atomics


def test_all_plus_signs_is_low_rank_product():
    # With every sign +1 the layer collapses to a rank-l chain whose l x l core can be
    # ill-conditioned, so a coherent rounding of V is amplified instead of averaged out;
    # bf16 envelopes keep the kernel's private bf16 copy of V exact.
    spec = small_spec(d_out=96, d_in=256, k=128, l=4, env_dtype="bf16", outliers=False)
    lay = inputs.make_layer(spec)
    lay["S_A"] = np.ones_like(lay["S_A"])
    lay["S_B"] = np.ones_like(lay["S_B"])
    x = inputs.make_activations(spec, 1)
    with GpuLayer(spec, 1, lay=lay) as g:
        ref = (np.linalg.multi_dot([lay["U_A"].astype(np.float64), lay["V_A"].T.astype(np.float64),
                                    lay["U_B"].astype(np.float64), lay["V_B"].T.astype(np.float64)])
               @ x.T.astype(np.float64)).T
        assert rel_err(g.forward(x), ref) <= TOL["bf16"]


# ------------------------------------------------- oracle-free properties
def test_linearity_column_independence_and_duality():
    spec = small_spec(d_out=256, d_in=384, k=256, l=16, outliers=False)
    lay = inputs.make_layer(spec)
    x4 = inputs.make_activations(spec, 4)
    with GpuLayer(spec, 4, lay=lay) as g:
        y4 = g.forward(x4)
        for t in (0, 2):                       # T-batched equals per-column (same kernel variant: exact)
            assert rel_err(g.forward(x4[t:t + 2]), y4[t:t + 2]) <= 1e-6
        for t in range(4):                     # one token may take another variant: equal within rounding
            assert rel_err(g.forward(x4[t:t + 1]), y4[t:t + 1]) <= 2 * TOL["bf16"]
        # linearity: power-of-two scaling is exact in bf16/fp32 arithmetic
        y_scaled = g.forward(4.0 * x4)
        np.testing.assert_array_equal(y_scaled, 4.0 * y4)
        # additivity within rounding
        xs = inputs.round_to(x4[0:1] + x4[1:2], "bf16")
        assert rel_err(g.forward(xs), (y4[0:1] + y4[1:2])) <= 2 * TOL["bf16"]
    # transpose duality: u^T (W v) = (W^T u)^T v with the factor roles swapped
    specT = inputs.scaled(spec, d_out=spec.d_in, d_in=spec.d_out)
    layT = {"S_A": lay["S_B"].T.copy(), "S_B": lay["S_A"].T.copy(), "U_A": lay["V_B"], "V_A": lay["U_B"],
            "U_B": lay["V_A"], "V_B": lay["U_A"]}
    rng = np.random.default_rng(9)
    u = inputs.round_to(rng.standard_normal((1, spec.d_out)), "bf16")
    v = inputs.round_to(rng.standard_normal((1, spec.d_in)), "bf16")
    with GpuLayer(spec, 1, lay=lay) as g, GpuLayer(specT, 1, lay=layT) as gT:
        lhs = (u.astype(np.float64) @ g.forward(v).T.astype(np.float64)).item()
        rhs = (gT.forward(u).astype(np.float64) @ v.T.astype(np.float64)).item()
        scale = np.linalg.norm(u) * np.linalg.norm(g.forward(v))
        assert abs(lhs - rhs) <= 2 * TOL["bf16"] * scale


# ------------------------------------------------------------- error paths
def test_forward_error_paths():
    spec = small_spec(d_out=64, d_in=128, k=64, l=4)
    with GpuLayer(spec, 2) as g:
        x = torch.zeros((4, 128), dtype=torch.bfloat16, device="cuda")
        y = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
        for T, dt, status in [(0, M.BF16, M.ERR_SHAPE), (3, M.BF16, M.ERR_SHAPE), (1, 9, M.ERR_DTYPE)]:
            with pytest.raises(M.MdbfError) as e:
                M.mdbf_linear_forward(g.h, x.data_ptr(), y.data_ptr(), T, dt)
            assert e.value.status == status
        with pytest.raises(M.MdbfError) as e:
            M.mdbf_linear_forward(g.h, 0, y.data_ptr(), 1, M.BF16)
        assert e.value.status == M.ERR_INVALID_ARG
        with pytest.raises(M.MdbfError) as e:
            M.mdbf_set_kernel(g.h, 17)
        assert e.value.status == M.ERR_INVALID_ARG
        assert M.mdbf_poll_status(g.h) == 0
    # fp32 envelopes cannot take the tensor-core kernels
    spec32 = inputs.scaled(inputs.tiny(), act_dtype="bf16")
    with GpuLayer(spec32, 1) as g:
        xb = inputs.round_to(inputs.make_activations(spec32, 1), "bf16")
        with pytest.raises(M.MdbfError) as e:
            g.forward(xb, kernel=M.KERNEL_TMEM)
        assert e.value.status == M.ERR_DTYPE
        assert rel_err(g.forward(xb), g.oracle_forward(xb)) <= TOL["bf16"]     # AUTO -> fp32 path


def test_host_buffer_entry_point():
    spec = small_spec()
    x = inputs.make_activations(spec, 2)
    with GpuLayer(spec, 2) as g:
        xh = torch.from_numpy(x).to(torch.bfloat16).pin_memory()
        yh = torch.zeros((2, spec.d_out), dtype=torch.bfloat16).pin_memory()
        with pytest.raises(M.MdbfError) as e:                      # no staging buffers yet: the call never allocates
            M.mdbf_linear_forward_host(g.h, xh.data_ptr(), yh.data_ptr(), 2, M.BF16, torch.cuda.current_stream().cuda_stream)
        assert e.value.status == M.ERR_INVALID_ARG
        M.mdbf_prepare_host_staging(g.h)
        M.mdbf_linear_forward_host(g.h, xh.data_ptr(), yh.data_ptr(), 2, M.BF16,
                                   torch.cuda.current_stream().cuda_stream)
        y_dev = g.forward(x)
        np.testing.assert_array_equal(yh.to(torch.float32).numpy(), y_dev)
        # without the final synchronisation: valid once the caller has synchronised the stream
        yh.zero_()
        st = torch.cuda.current_stream().cuda_stream
        M.mdbf_linear_forward_host_async(g.h, xh.data_ptr(), yh.data_ptr(), 2, M.BF16, st)
        M.mdbf_linear_forward_host_async(g.h, xh.data_ptr(), yh.data_ptr(), 2, M.BF16, st)   # same handle: ordered by the stream
        torch.cuda.current_stream().synchronize()
        np.testing.assert_array_equal(yh.to(torch.float32).numpy(), y_dev)
