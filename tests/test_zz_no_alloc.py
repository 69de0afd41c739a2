"""The workspace-free decode entry point, for hosts that cannot allocate device memory.

templora_decode_fwd_noalloc keeps its scratch in a fixed array inside the library instead of a
caller-provided workspace.  It must give the same output as templora_decode_fwd, call after call
(the array is shared and keeps the previous call's contents), and must refuse a projection whose
scratch would not fit.  This file sorts last on purpose: a run that stops at the first failure
has then already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2401_11504_b200 import inputs
from parity_utils import TOL, assert_close, f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2401_11504_b200 import build
    build.build_library()
    from paper_2401_11504_b200 import binding
    binding.templora_set_kernel_path(0)
    return binding


def _case(b, seed, n, d_in, d_out, r, dtype="bf16"):
    host = inputs.make_linear(seed, f"noalloc-{n}-{d_in}-{d_out}", n, d_in, d_out, r, dtype=dtype)
    dev = {k: v.cuda() for k, v in host.items()}
    lin = b.linear_desc(dev["W0"], dev["A"], dev["B"], 2.0)
    ws = b.alloc_workspace(b.templora_workspace_bytes(lin, 16))
    want = torch.empty((n, d_out), dtype=host["x"].dtype, device="cuda")
    b.templora_decode_fwd(lin, dev["x"], want, ws)
    torch.cuda.synchronize()
    return lin, dev["x"], want


def test_two_calls_in_a_row_match_the_workspace_entry_point(b):
    # two different projections back to back: the second call finds the first one's leftovers
    # in the shared array and must not be disturbed by them
    cases = [_case(b, 31, 16, 4096, 1024, 64), _case(b, 32, 4, 1024, 2048, 16)]
    for lin, x, want in cases:
        got = torch.full_like(want, float("nan"))
        b.templora_decode_fwd_noalloc(lin, x, got)
        torch.cuda.synchronize()
        assert_close("noalloc decode", f64(got), f64(want), TOL["bf16"])
        assert np.abs(f64(want)).max() > 0
    # and the first one again, after the array has held another shape's partial sums
    lin, x, want = cases[0]
    got = torch.full_like(want, float("nan"))
    b.templora_decode_fwd_noalloc(lin, x, got)
    torch.cuda.synchronize()
    assert_close("noalloc decode (repeat)", f64(got), f64(want), TOL["bf16"])


def test_generic_path_shapes_work_too(b):
    lin, x, want = _case(b, 33, 3, 100, 60, 4, dtype="f32")
    got = torch.full_like(want, float("nan"))
    b.templora_decode_fwd_noalloc(lin, x, got)
    torch.cuda.synchronize()
    assert_close("noalloc decode fp32", f64(got), f64(want), TOL["f32"])


def test_oversize_projection_is_refused(b):
    # one k-block, 262144 output rows: 16 * d_out fp32 partial sums alone are 16 MiB > 8 MiB
    d_in, d_out, r = 64, 262144, 8
    W0 = torch.zeros((d_out, d_in), dtype=torch.bfloat16, device="cuda")
    A = torch.zeros((r, d_in), dtype=torch.bfloat16, device="cuda")
    B = torch.zeros((d_out, r), dtype=torch.bfloat16, device="cuda")
    lin = b.linear_desc(W0, A, B, 2.0)
    x = torch.zeros((16, d_in), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((16, d_out), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(b.TemploraError) as e:
        b.templora_decode_fwd_noalloc(lin, x, y)
    assert e.value.code == b.ERR_UNSUPPORTED
    with pytest.raises(b.TemploraError) as e:
        b.templora_decode_fwd_noalloc(lin, torch.zeros((17, d_in), dtype=torch.bfloat16, device="cuda"), y)
    assert e.value.code == b.ERR_INVALID_ARG
