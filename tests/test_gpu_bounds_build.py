"""The bounds-checked build of the library (MDBF_BOUNDS_CHECK=1 in the environment of the test run): the same GPU
suite runs against it, every forward of the helpers reads the status word, and this file checks that the variant
that was asked for is the one that got loaded."""
import os

import pytest
import torch

from paper_2512_24545_b200 import inputs, mdbf as M
from helpers import GpuLayer, check_parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2512_24545_b200 import build
    build.build()
    assert torch.cuda.is_available()


def test_loaded_library_is_the_requested_variant():
    want = os.environ.get("MDBF_BOUNDS_CHECK", "0") not in ("", "0")
    assert ("+bounds-check" in M.version()) == want


@pytest.mark.parametrize("T", [1, 7, 300])
def test_forward_between_guard_regions_leaves_status_clean(T):
    """Ragged in every dimension: the last row block, K block and token tile are partial.  GpuLayer.forward puts y
    between two guard regions and asserts that they are untouched and that the status word reads 0."""
    spec = inputs.scaled(inputs.qproj(1664), name="guard", d_out=333, d_in=520, k=190, l=16, outliers=False)
    x = inputs.make_activations(spec, T)
    with GpuLayer(spec, max(T, 2)) as g:                       # the expanded order needs a handle packed for T >= 2
        for kernel in (M.KERNEL_AUTO, M.KERNEL_ALU, M.KERNEL_PREFILL) + ((M.KERNEL_I8, M.KERNEL_TMEM) if T == 1 else (M.KERNEL_MAT,)):
            y = g.forward(x, kernel=kernel)
            check_parity(g, x, y, roundings=4)
