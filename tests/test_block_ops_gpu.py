"""Parity of the SiLU gating and RMSNorm kernels (forward and backward) with the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import templora_oracle as orc
from paper_2401_11504_b200 import inputs
from parity_utils import TOL, assert_close, f64, tdtype

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2401_11504_b200 import build
    build.build_library()
    from paper_2401_11504_b200 import binding
    return binding


def _t(seed, tag, shape, dtype, scale=1.0):
    return inputs.make_tensor(seed, "blockops", tag, shape, "normal", scale, dtype, "cuda")


# shapes: the 7B MLP width, a ragged width (scalar tail / unaligned rows), tiny
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("T,d", [(64, 11008), (37, 1000), (5, 7), (1, 8)])
def test_swiglu_matches_oracle(b, dtype, T, d):
    g, u, dh = (_t(40, f"{n}-{T}-{d}", (T, d), dtype, 2.0) for n in ("g", "u", "dh"))
    h = torch.full_like(g, float("nan"))
    b.templora_swiglu_fwd(g, u, h)
    assert_close("h", f64(h), orc.swiglu_fwd(f64(g), f64(u)), TOL[dtype])
    dg, du = torch.full_like(g, float("nan")), torch.full_like(g, float("nan"))
    b.templora_swiglu_bwd(g, u, dh, dg, du)
    rg, ru = orc.swiglu_bwd(f64(g), f64(u), f64(dh))
    assert_close("dgate", f64(dg), rg, TOL[dtype])
    assert_close("dup", f64(du), ru, TOL[dtype])


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("T,d", [(130, 4096), (16, 11008), (9, 1000), (3, 100), (2, 5)])
def test_rmsnorm_matches_oracle(b, dtype, T, d):
    x, dy = _t(41, f"x-{T}-{d}", (T, d), dtype, 3.0), _t(41, f"dy-{T}-{d}", (T, d), dtype)
    w = inputs.make_tensor(41, "blockops", f"w-{d}", (d,), "uniform", 1.5, dtype, "cuda")
    eps = float(np.float32(1e-5))
    y, dx = torch.full_like(x, float("nan")), torch.full_like(x, float("nan"))
    b.templora_rmsnorm_fwd(x, w, eps, y)
    assert_close("y", f64(y), orc.rmsnorm_fwd(f64(x), f64(w), eps), TOL[dtype])
    b.templora_rmsnorm_bwd(x, w, dy, eps, dx)
    assert_close("dx", f64(dx), orc.rmsnorm_bwd(f64(x), f64(w), f64(dy), eps), TOL[dtype])


def test_rmsnorm_row_by_row_tolerance_fp32(b):
    # rows of very different scale: the check is per row, so a wrong rstd on a small row cannot hide
    T, d = 8, 512
    x = _t(42, "xs", (T, d), "f32") * torch.logspace(-3, 3, T, device="cuda").unsqueeze(1)
    w = torch.ones(d, device="cuda")
    y = torch.empty_like(x)
    b.templora_rmsnorm_fwd(x.contiguous(), w, 0.0, y)
    ref = orc.rmsnorm_fwd(f64(x), f64(w), 0.0)
    for t in range(T):
        assert_close(f"row {t}", f64(y)[t], ref[t], TOL["f32"])


def test_block_ops_reject_bad_arguments(b):
    x = torch.zeros((4, 16), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(b.TemploraError):
        b.templora_rmsnorm_fwd(x, x[0], -1.0, x)          # negative eps
    with pytest.raises(b.TemploraError):
        b.templora_swiglu_fwd(x.flatten()[1:9], x.flatten()[1:9], x.flatten()[1:9])   # not 16-byte aligned
