"""The workspace-free decode entry point, for hosts that cannot allocate device memory.

templora_decode_fwd_noalloc keeps its scratch in a fixed array inside the library instead of a
caller-provided workspace.  It must give the same output as templora_decode_fwd (and as the fp64
oracle), call after call (the array is shared and keeps the previous call's contents), in every
kernel form the decode path has, and must refuse a projection whose scratch would not fit.  This
file sorts last on purpose: a run that stops at the first failure has then already run every
other test.
"""
import numpy as np
import pytest
import torch

from oracle import templora_oracle as orc
from paper_2401_11504_b200 import inputs
from parity_utils import TOL, assert_close, f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2401_11504_b200 import build
    build.build_library()
    from paper_2401_11504_b200 import binding
    binding.templora_set_kernel_path(0)
    yield binding
    binding.templora_set_kernel_path(0)


def _case(b, seed, n, d_in, d_out, r, dtype="bf16"):
    """-> (descriptor, x, output of the workspace entry point, the oracle's output)."""
    host = inputs.make_linear(seed, f"noalloc-{n}-{d_in}-{d_out}", n, d_in, d_out, r, dtype=dtype)
    dev = {k: v.cuda() for k, v in host.items()}
    lin = b.linear_desc(dev["W0"], dev["A"], dev["B"], 2.0)
    ws = b.alloc_workspace(b.templora_workspace_bytes(lin, 16))
    want = torch.empty((n, d_out), dtype=host["x"].dtype, device="cuda")
    b.templora_decode_fwd(lin, dev["x"], want, ws)
    torch.cuda.synchronize()
    ref = orc.decode_fwd(f64(host["x"]), f64(host["W0"]), f64(host["A"]), f64(host["B"]), 2.0)
    return lin, dev["x"], want, ref


def _run_and_check(b, what, lin, x, want, ref, tol):
    got = torch.full_like(want, float("nan"))
    b.templora_decode_fwd_noalloc(lin, x, got)
    assert b.templora_decode_fwd_noalloc_status() == (0, 0)      # synchronises; no bounded wait ran out
    assert_close(f"{what}: against the oracle", f64(got), ref, tol)
    assert_close(f"{what}: against templora_decode_fwd", f64(got), f64(want), tol)
    assert np.abs(ref).max() > 0


# kernel path 0: the one-kernel cluster form; path 2: the W0 stream with split-K partial slabs in the array
# plus the finishing kernel (the form whose leftovers from an earlier call of another shape matter)
@pytest.mark.parametrize("path", [0, 2])
def test_two_calls_in_a_row_match_the_workspace_entry_point(b, path):
    b.templora_set_kernel_path(path)
    try:
        # different projections back to back: each call finds the previous one's leftovers in the shared
        # array (other slab sizes, other token counts) and must not be disturbed by them
        cases = [_case(b, 31, 16, 4096, 1024, 64), _case(b, 32, 4, 1024, 2048, 16), _case(b, 34, 7, 2048, 640, 32)]
        for k, (lin, x, want, ref) in enumerate(cases):
            _run_and_check(b, f"path {path} call {k}", lin, x, want, ref, TOL["bf16"])
        # and the first one again, after the array has held other shapes' partial sums
        lin, x, want, ref = cases[0]
        _run_and_check(b, f"path {path} repeat", lin, x, want, ref, TOL["bf16"])
    finally:
        b.templora_set_kernel_path(0)


@pytest.mark.parametrize("cap", [8, 1])
def test_under_a_tight_sm_cap(b, cap):
    # with few SMs allowed on the stream the cluster form runs on few clusters (cap 8) or gives way to the
    # two-kernel form (cap 1: no cluster fits)
    stream = torch.cuda.current_stream()
    cases = [_case(b, 35, 16, 2048, 1024, 64), _case(b, 36, 1, 1024, 512, 16)]
    b.templora_set_stream_sm_limit(stream, cap)
    try:
        for k, (lin, x, want, ref) in enumerate(cases + cases[:1]):
            _run_and_check(b, f"cap {cap} call {k}", lin, x, want, ref, TOL["bf16"])
    finally:
        b.templora_set_stream_sm_limit(stream, 0)


def test_generic_path_shapes_work_too(b):
    lin, x, want, ref = _case(b, 33, 3, 100, 60, 4, dtype="f32")
    _run_and_check(b, "fp32", lin, x, want, ref, TOL["f32"])


def test_refusals_enqueue_nothing(b):
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
    # the same codes as templora_decode_fwd for a rank beyond 256 and for a misaligned input
    big_r = b.linear_desc(torch.zeros((64, 64), dtype=torch.bfloat16, device="cuda"),
                          torch.zeros((264, 64), dtype=torch.bfloat16, device="cuda"),
                          torch.zeros((64, 264), dtype=torch.bfloat16, device="cuda"), 2.0)
    with pytest.raises(b.TemploraError) as e:
        b.templora_decode_fwd_noalloc(big_r, x, y)
    assert e.value.code == b.ERR_UNSUPPORTED
    small = b.linear_desc(W0[:64].contiguous(), A, B[:64].contiguous(), 2.0)
    with pytest.raises(b.TemploraError) as e:
        b.templora_decode_fwd_noalloc(small, x.view(-1)[1:1 + 64].view(1, 64), y)
    assert e.value.code == b.ERR_INVALID_ARG
    assert b.templora_decode_fwd_noalloc_status() == (0, 0)
