"""The seeded generators: determinism, storage-type representability, recipe."""
import numpy as np
import torch

from paper_2512_24545_b200 import inputs


def test_layer_is_deterministic_and_representable():
    spec = inputs.scaled(inputs.qproj(1664), d_out=96, d_in=160, k=64)
    a, b = inputs.make_layer(spec), inputs.make_layer(spec)
    for key in a:
        np.testing.assert_array_equal(a[key], b[key])
    assert set(np.unique(a["S_A"])) == {-1, 1} and a["S_A"].dtype == np.int8
    assert a["S_A"].shape == (96, 64) and a["S_B"].shape == (64, 160)
    for key in ("U_A", "V_A", "U_B", "V_B"):
        v = torch.from_numpy(a[key])
        assert torch.equal(v.to(torch.float16).to(torch.float32), v)       # fp16 values
    assert abs(float(np.std(a["V_B"])) - 0.02) < 0.004
    assert abs(float(np.mean(a["S_B"] == -1)) - 0.5) < 0.03


def test_activations_recipe():
    spec = inputs.scaled(inputs.qproj(1664), d_in=2000)
    x4 = inputs.make_activations(spec, 4)
    assert x4.shape == (4, 2000) and x4.dtype == np.float32
    v = torch.from_numpy(x4)
    assert torch.equal(v.to(torch.bfloat16).to(torch.float32), v)          # bf16 values
    col_rms = np.sqrt(np.mean(x4.astype(np.float64) ** 2, axis=0))
    assert int(np.sum(col_rms > 6.0)) == 20                                # 1 % outlier channels x20
    np.testing.assert_array_equal(inputs.make_activations(spec, 4), x4)
    plain = inputs.make_activations(inputs.scaled(spec, outliers=False), 4)
    assert np.max(np.abs(plain)) < 6.0


def test_tiny_config_is_fp32():
    spec = inputs.tiny()
    lay = inputs.make_layer(spec)
    assert lay["U_A"].shape == (256, 4) and lay["V_A"].shape == (128, 4)
    assert abs(float(np.std(lay["U_B"])) - 128 ** -0.5) < 0.02
    x = inputs.make_activations(spec, 8)
    assert x.shape == (8, 256)
    # fp32 storage: values are not generally bf16-representable
    v = torch.from_numpy(x)
    assert not torch.equal(v.to(torch.bfloat16).to(torch.float32), v)


def test_block_specs():
    specs = inputs.block70b()
    assert [s.name.split("_")[1] for s in specs] == ["q", "k", "v", "o", "gate", "up", "down"]
    assert len({s.seed for s in specs}) == 7
    assert specs[4].d_out == 28672 and specs[6].d_in == 28672 and specs[1].k == 512
