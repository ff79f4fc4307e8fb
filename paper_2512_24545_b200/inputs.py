"""Seeded synthetic inputs for the MDBF linear forward.

This module only draws random numbers and rounds them to their storage type;
it holds none of the method's arithmetic.  Both the CPU oracle's tests and the
CUDA path's tests/bench take their data from here, so that the two sides see
bit-identical stored values.

The shapes stand in for the projection shapes of the 7B- and 70B-class
decoder models the paper quantizes (its trained weights and evaluation text
are not used anywhere): i.i.d. Bernoulli(1/2) signs, Gaussian envelope factors
rounded to fp16 (fp32 for the tiny case), Gaussian activations rounded to bf16
with 1 % of the input channels scaled by 20 ("outlier channels") where the
workload says so.

Random streams: numpy PCG64 seeded from SeedSequence(seed).spawn(8), in the
fixed order  [S_A, S_B, U_A, V_A, U_B, V_B, x, outlier-index].
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List

import numpy as np
import torch

_STREAMS = ("S_A", "S_B", "U_A", "V_A", "U_B", "V_B", "x", "outlier")


@dataclass(frozen=True)
class LayerSpec:
    name: str
    d_out: int
    d_in: int
    k: int
    l: int
    seed: int
    env_dtype: str = "f16"      # storage type of U_A, V_A, U_B, V_B: "f32" | "f16" | "bf16"
    act_dtype: str = "bf16"     # type of x and y: "f32" | "bf16"
    env_std: float = 0.02       # standard deviation of the envelope entries
    outliers: bool = True       # 1 % outlier input channels x20


def _rng(seed: int, stream: str) -> np.random.Generator:
    child = np.random.SeedSequence(seed).spawn(len(_STREAMS))[_STREAMS.index(stream)]
    return np.random.Generator(np.random.PCG64(child))


def round_to(a: np.ndarray, dtype: str) -> np.ndarray:
    """Round float values to `dtype` (round-to-nearest-even) and return them as float32."""
    a32 = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "f32":
        return a32
    tdt = {"f16": torch.float16, "bf16": torch.bfloat16}[dtype]
    return torch.from_numpy(a32).to(tdt).to(torch.float32).numpy()


def make_signs(rows: int, cols: int, seed: int, stream: str) -> np.ndarray:
    bits = _rng(seed, stream).integers(0, 2, size=(rows, cols), dtype=np.int8)
    return (1 - 2 * bits).astype(np.int8)          # bit 1 -> -1, bit 0 -> +1


def make_layer(spec: LayerSpec) -> Dict[str, np.ndarray]:
    """Signs (int8 +-1) and envelope factors (float32 holding values already
    rounded to spec.env_dtype)."""
    out = {
        "S_A": make_signs(spec.d_out, spec.k, spec.seed, "S_A"),
        "S_B": make_signs(spec.k, spec.d_in, spec.seed, "S_B"),
    }
    shapes = {"U_A": (spec.d_out, spec.l), "V_A": (spec.k, spec.l),
              "U_B": (spec.k, spec.l), "V_B": (spec.d_in, spec.l)}
    for name, shp in shapes.items():
        g = _rng(spec.seed, name).standard_normal(shp) * spec.env_std
        out[name] = round_to(g, spec.env_dtype)
    return out


def make_activations(spec: LayerSpec, T: int, seed_offset: int = 0) -> np.ndarray:
    """x as a (T, d_in) float32 array (token-contiguous) holding values already
    rounded to spec.act_dtype."""
    seed = spec.seed + seed_offset
    x = _rng(seed, "x").standard_normal((T, spec.d_in))
    if spec.outliers:
        n_out = int(round(0.01 * spec.d_in))
        ch = _rng(seed, "outlier").choice(spec.d_in, size=n_out, replace=False)
        x[:, ch] *= 20.0
    return round_to(x, spec.act_dtype)


# ---------------------------------------------------------------------------
# The five workloads.  Inner ranks k are the largest multiples of 128 that
# meet the stated bits-per-weight budget with 16-bit envelopes; the table is
# written out here (data), and tests check it against the oracle's accounting.
# ---------------------------------------------------------------------------
def tiny() -> LayerSpec:
    k = 128
    return LayerSpec("tiny", 256, 256, k, 4, seed=0, env_dtype="f32", act_dtype="f32",
                     env_std=float(k) ** -0.5, outliers=False)


def qproj(k: int) -> LayerSpec:
    assert k in (1664, 2560)
    return LayerSpec(f"q_proj_k{k}", 4096, 4096, k, 16, seed=2)


def mlp(which: str) -> LayerSpec:
    if which in ("up", "gate"):
        return LayerSpec(f"mlp_{which}", 11008, 4096, 3968, 16, seed=3)
    assert which == "down"
    return LayerSpec("mlp_down", 4096, 11008, 3968, 16, seed=3)


PREFILL_K = {  # (d_out, d_in, l) -> (k at ~1.0 bpw, k at ~1.5 bpw)
    (4096, 4096, 1): (1920, 2944), (4096, 4096, 4): (1920, 2944), (4096, 4096, 16): (1664, 2560),
    (11008, 4096, 1): (2944, 4352), (11008, 4096, 4): (2816, 4352), (11008, 4096, 16): (2560, 3968),
}


def prefill(d_out: int, l: int, bpw: float) -> LayerSpec:
    k = PREFILL_K[(d_out, 4096, l)][0 if bpw < 1.25 else 1]
    return LayerSpec(f"prefill_{d_out}x4096_l{l}_k{k}", d_out, 4096, k, l, seed=4, outliers=False)


BLOCK70B = (  # name, d_out, d_in, k   (l = 16, ~1.0 bpw)
    ("q", 8192, 8192, 3712), ("k", 1024, 8192, 512), ("v", 1024, 8192, 512),
    ("o", 8192, 8192, 3712), ("gate", 28672, 8192, 6016), ("up", 28672, 8192, 6016),
    ("down", 8192, 28672, 6016),
)


def block70b() -> List[LayerSpec]:
    return [LayerSpec(f"block70b_{n}", do, di, k, 16, seed=5 + 1000 * idx)
            for idx, (n, do, di, k) in enumerate(BLOCK70B)]


def scaled(spec: LayerSpec, **kw) -> LayerSpec:
    """A copy of `spec` with some fields replaced (reduced shapes for quick tests)."""
    return replace(spec, **kw)


# ---------------------------------------------------------------- inputs of the quantizer's first step
def make_factor_matrix(rows: int, cols: int, seed: int, special_values: bool = True) -> np.ndarray:
    """A dense fp32 matrix to hand to the Multi-Envelope SVID: Gaussian entries under log-normal row and column
    scales (the envelope of a trained factor is not flat), a few exact zeros, a negative zero and a tiny negative
    entry so that the sign convention sign(0) = +1 is exercised.  Stands in for the balanced SVD factors of a
    checkpoint's weight matrix, which are not available here."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, rows, cols])))
    Z = rng.standard_normal((rows, cols))
    Z *= np.exp(0.5 * rng.standard_normal((rows, 1))) * np.exp(0.5 * rng.standard_normal((1, cols)))
    Z = Z.astype(np.float32)
    if special_values and rows * cols >= 8:
        flat = Z.reshape(-1)
        idx = rng.choice(flat.size, size=min(8, flat.size), replace=False)
        flat[idx[:-2]] = 0.0
        flat[idx[-2]] = -0.0
        flat[idx[-1]] = -1e-30
    return Z


def make_start_block(cols: int, l: int, seed: int) -> np.ndarray:
    """The cols x l Gaussian block a subspace iteration starts from (drawn here, passed in as an input)."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, cols, l, 7])))
    return rng.standard_normal((cols, l)).astype(np.float32)
