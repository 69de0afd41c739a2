"""CPU-only checks of the C-ABI library: it builds, loads, exports every symbol the public
header declares, and its host-side argument checks answer without touching a GPU."""
import ctypes as C
import os
import re

import pytest

from conftest import ROOT


@pytest.fixture(scope="module")
def b():
    from paper_2401_11504_b200 import build
    build.build_library()
    from paper_2401_11504_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "templora.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(templora_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(b):
    names = declared_functions()
    assert len(names) >= 10
    raw = C.CDLL(b.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), f"{n} declared in templora.h but not exported"
    assert sorted(b.EXPORTS) == [n for n in names if n in b.EXPORTS]
    for n in names:
        assert n in b.EXPORTS, f"{n} has no Python binding"


def test_status_strings(b):
    seen = {b.status_string(c) for c in range(6)}
    assert len(seen) == 6 and "ok" in seen
    assert b.status_string(99) == "unknown status"


def _lin(b, d_in=4096, d_out=4096, r=64, dtype=None, ptr=0x1000):
    return b.LinearDesc(d_in, d_out, r, 2.0, b.BF16 if dtype is None else dtype, ptr, ptr, ptr)


def test_workspace_sizes_are_sane(b):
    lin = _lin(b)
    n1 = b.templora_workspace_bytes(lin, 1024)
    n2 = b.templora_workspace_bytes(lin, 2048)
    assert 1024 < n1 < n2 < (1 << 30)
    assert b.templora_workspace_bytes(lin, 0) == 0
    assert b.templora_workspace_bytes(_lin(b, r=512), 128) == 0          # rank beyond 256
    assert b.templora_workspace_bytes(_lin(b, dtype=7), 128) == 0
    from paper_2401_11504_b200 import inputs
    lins = [_lin(b, di, do) for _, di, do in inputs.LLAMA2_7B_BLOCK]
    nb = b.templora_update_block_workspace_bytes(lins, 1024)
    assert n1 <= nb < (1 << 31)
    # a block of 32 x 7 projections needs no more than the largest group of 8
    assert b.templora_update_block_workspace_bytes(lins * 32, 1024) <= 2 * nb


def test_noalloc_scratch_holds_every_7b_and_70b_projection(b):
    # the header promises that the built-in array of templora_decode_fwd_noalloc is large enough for every
    # Llama-2 7B- and 70B-shaped projection at rank 64 with up to 16 tokens, in either decode kernel form
    from paper_2401_11504_b200 import inputs
    lib = b.lib
    assert b.NOALLOC_SCRATCH_BYTES == 8 << 20
    worst = 0
    for block in (inputs.LLAMA2_7B_BLOCK, inputs.LLAMA2_70B_BLOCK):
        for name, d_in, d_out in block:
            need = b.templora_decode_block_workspace_bytes([_lin(b, d_in, d_out, 64)])
            assert 1024 <= need <= b.NOALLOC_SCRATCH_BYTES, (name, d_in, d_out, need)
            worst = max(worst, need)
    assert worst > (1 << 20)     # the query really measures the split-K slabs, not just the head
    # refusals need no GPU: token count, rank, missing tensors
    lin = _lin(b)
    vp = C.c_void_p
    assert lib.templora_decode_fwd_noalloc(C.byref(lin), 17, vp(0x1000), vp(0x1000), None) == b.ERR_INVALID_ARG
    assert lib.templora_decode_fwd_noalloc(C.byref(lin), 4, None, vp(0x1000), None) == b.ERR_INVALID_ARG
    assert lib.templora_decode_fwd_noalloc(C.byref(_lin(b, r=257)), 4, vp(0x1000), vp(0x1000), None) == b.ERR_UNSUPPORTED
    assert lib.templora_decode_fwd_noalloc(C.byref(_lin(b, 64, 1 << 18, 8)), 16, vp(0x1000), vp(0x1000), None) == b.ERR_UNSUPPORTED
    assert lib.templora_decode_fwd_noalloc_status(None, None, None) == b.ERR_INVALID_ARG


def test_argument_errors_are_synchronous(b):
    lib = b.lib
    lin = _lin(b)
    vp = C.c_void_p
    # NULL tensors, zero rows, bad token counts, missing workspace: all rejected before any launch
    assert lib.templora_linear_fwd(C.byref(lin), 16, None, None, None, None, 0, None) == b.ERR_INVALID_ARG
    assert lib.templora_linear_fwd(C.byref(lin), 0, vp(0x1000), vp(0x1000), None, vp(0x1000), 1 << 20, None) == b.ERR_INVALID_ARG
    assert lib.templora_linear_fwd(C.byref(lin), 16, vp(0x1008), vp(0x1000), None, vp(0x1000), 1 << 20, None) == b.ERR_INVALID_ARG
    assert lib.templora_linear_fwd(C.byref(lin), 16, vp(0x1000), vp(0x1000), None, None, 0, None) == b.ERR_WORKSPACE
    assert lib.templora_linear_fwd(C.byref(lin), 16, vp(0x1000), vp(0x1000), None, vp(0x1010), 1 << 20, None) == b.ERR_WORKSPACE
    assert lib.templora_decode_fwd(C.byref(lin), 17, vp(0x1000), vp(0x1000), vp(0x1000), 1 << 20, None) == b.ERR_INVALID_ARG
    assert lib.templora_decode_fwd(C.byref(lin), 0, vp(0x1000), vp(0x1000), vp(0x1000), 1 << 20, None) == b.ERR_INVALID_ARG
    bad = _lin(b, r=257)
    assert lib.templora_linear_fwd(C.byref(bad), 16, vp(0x1000), vp(0x1000), None, vp(0x1000), 1 << 20, None) == b.ERR_UNSUPPORTED
    assert lib.templora_linear_bwd(C.byref(lin), 16, vp(0x1000), vp(0x1000), None, None, None, None, 0,
                                   vp(0x1000), 1 << 20, None) == b.ERR_INVALID_ARG
    p = b.ParamDesc(16, 0x1000, 0x1000, 0x1000, 0, 0x1000)
    arr = (b.ParamDesc * 1)(p)
    assert lib.templora_adamw_step(arr, 1, 1e-3, 0.9, 0.999, 1e-8, 0.0, 0, b.BF16, None) == b.ERR_INVALID_ARG   # step < 1
    assert lib.templora_adamw_step(arr, 1, 1e-3, 1.5, 0.999, 1e-8, 0.0, 1, b.BF16, None) == b.ERR_INVALID_ARG   # beta1
    assert lib.templora_adamw_step(None, 1, 1e-3, 0.9, 0.999, 1e-8, 0.0, 1, b.BF16, None) == b.ERR_INVALID_ARG


def test_update_block_rejects_unaliased_parameters(b):
    lib = b.lib
    lin = _lin(b, ptr=0x2000)
    lins = (b.LinearDesc * 1)(lin)
    A = (b.ParamDesc * 1)(b.ParamDesc(64 * 4096, 0x1000, 0x1000, 0x1000, 0x3000, 0x1000))   # work != lin.A
    Bp = (b.ParamDesc * 1)(b.ParamDesc(64 * 4096, 0x1000, 0x1000, 0x1000, 0x2000, 0x1000))
    vp = C.c_void_p
    arr = (vp * 1)(0x1000)
    step = C.c_int64(0)
    rc = lib.templora_update_block(lins, A, Bp, 1, 16, arr, arr, arr, None, 1, 1e-3, 0.9, 0.999, 1e-8, 0.0,
                                   C.byref(step), vp(0x1000), 1 << 20, None)
    assert rc == b.ERR_INVALID_ARG and step.value == 0


def test_kernel_path_switch_round_trips(b):
    prev = b.templora_set_kernel_path(1)
    assert b.templora_set_kernel_path(prev) == 1


def test_lr_at_step_host_function(b):
    # host arithmetic only: same closed form as the oracle's, in fp32
    import numpy as np
    from oracle import templora_oracle as orc
    lr = float(np.float32(5e-5))
    for step, w in ((1, 8), (4, 8), (8, 8), (9, 8), (5, 0), (0, 4)):
        got = b.templora_lr_at_step(lr, step, w)
        assert got == float(np.float32(orc.lr_at_step(lr, step, w)))


def test_sm_partition_argument_errors_need_no_device(b):
    # refused before any driver call: nothing to split into, nowhere to put the result, nothing to destroy
    part = b.SmPartition()
    assert b.lib.templora_sm_partition_create(0, C.byref(part)) == b.ERR_INVALID_ARG
    assert b.lib.templora_sm_partition_create(32, None) == b.ERR_INVALID_ARG
    assert part.handle is None and part.stream_first is None and part.sms_first == 0
    assert b.lib.templora_sm_partition_destroy(C.byref(part)) == b.ERR_INVALID_ARG
    assert b.lib.templora_sm_partition_destroy(None) == b.ERR_INVALID_ARG
