"""templora_update_attn_in: the chunk update of the projections behind a decoder block's input norm (RMSNorm -> q, k, v
on the shared normalised input, one summed input gradient, the norm's backward) in one call, against a composition
of the oracle's functions (rmsnorm_fwd, update_block with shared inputs, rmsnorm_bwd: no arithmetic of its own here)."""
import numpy as np
import pytest
import torch

from oracle import templora_oracle as orc
from paper_2401_11504_b200 import inputs
from parity_utils import TOL, Guarded, assert_close, check_adam_steps, f64, hp32, ill_conditioned_mask, make_state

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2401_11504_b200 import build
    build.build_library()
    from paper_2401_11504_b200 import binding
    binding.templora_set_kernel_path(0)
    yield binding
    binding.templora_set_kernel_path(0)


def _attn_in_case(b, dtype, T, d, d_outs, r, epochs, seed, with_dX=True, norm_eps=1e-5):
    hp = hp32(dict(lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0))
    s = 2.0
    hosts = [inputs.make_linear(seed, f"attn{i}", T, d, do, r, dtype=dtype) for i, do in enumerate(d_outs)]
    x_h = hosts[0]["x"]
    w_h = inputs.make_tensor(seed, "attn", "norm_w", (d,), "uniform", 1.0, "bf16" if dtype == "bf16" else "f32", "cpu") + 1.0
    w_h = w_h.to(x_h.dtype)
    states = [make_state(h, dtype) for h in hosts]
    W0 = [h["W0"].cuda() for h in hosts]
    lins, As, Bs = [], [], []
    for w0, st in zip(W0, states):
        a = st["A"]["work"] if dtype == "bf16" else st["A"]["master"]
        bb = st["B"]["work"] if dtype == "bf16" else st["B"]["master"]
        lins.append(b.linear_desc(w0, a, bb, s))
        As.append(b.param_desc(st["A"]["master"], st["A"]["m"], st["A"]["v"], st["A"]["grad"], st["A"]["work"]))
        Bs.append(b.param_desc(st["B"]["master"], st["B"]["m"], st["B"]["v"], st["B"]["grad"], st["B"]["work"]))
    td = x_h.dtype
    guard = Guarded()
    xn, dXn = guard.empty((T, d), td), guard.empty((T, d), td)
    dX = guard.empty((T, d), td) if with_dX else None
    ys = [guard.empty((T, do), td) for do in d_outs]
    ws = guard.workspace(b.templora_update_block_workspace_bytes(lins, T))
    x, w = x_h.cuda(), w_h.cuda()
    dYs = [h["dY"].cuda() for h in hosts]
    step = b.templora_update_attn_in(lins, As, Bs, x, w, norm_eps, dYs, xn, ys, dXn, dX, epochs, hp["lr"], hp["beta1"],
                                     hp["beta2"], hp["eps"], hp["weight_decay"], 0, ws)
    assert step == epochs
    assert b.templora_read_device_status(ws) == (0, 0)
    guard.check("after templora_update_attn_in")

    # the oracle's composition: norm, projections on the shared normalised input with one summed gradient, norm backward
    xn_ref = orc.rmsnorm_fwd(f64(x_h), f64(w_h), norm_eps)
    projs = [dict(x=xn_ref, dY=f64(h["dY"]), W0=f64(h["W0"]), s=s, A_master=f64(h["A"]), B_master=f64(h["B"]),
                  dX_to=None if i == 0 else 0) for i, h in enumerate(hosts)]
    log = []
    ref, rstep = orc.update_block(projs, epochs, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"],
                                  bf16_work=(dtype == "bf16"), grad_log=log)
    assert rstep == epochs
    dX_ref = orc.rmsnorm_bwd(f64(x_h), f64(w_h), ref[0]["dX"], norm_eps)
    tol = TOL[dtype]
    assert_close("xn", f64(xn), xn_ref, tol)
    assert_close("dXn (summed over the projections)", f64(dXn), ref[0]["dX"], tol)
    if with_dX:
        assert_close("dX", f64(dX), dX_ref, tol)
    for i, (q, st) in enumerate(zip(ref, states)):
        assert_close(f"y{i}", f64(ys[i]), q["y"], tol)
        assert_close(f"dA{i}", f64(st["A"]["grad"]), q["dA"], tol)
        assert_close(f"dB{i}", f64(st["B"]["grad"]), q["dB"], tol)
        for P in ("A", "B"):
            p0 = f64(hosts[i][P])
            got = f64(st[P]["master"])
            mask = ill_conditioned_mask(log, i, P, p0, hp, tol)
            check_adam_steps(f"proj{i}.{P}", p0, got, q[P + "_master"], mask, tol, epochs, hp["lr"],
                             max_frac=0.03 if dtype == "bf16" else 1e-3)
            if dtype == "bf16":
                assert np.array_equal(f64(st[P]["work"]), orc.round_bf16(got.astype(np.float32)))


def test_attn_in_bf16_ragged_q_k_v(b):
    # grouped-query shapes: k, v narrower than q; rows not a multiple of any tile
    _attn_in_case(b, "bf16", 300, 512, (512, 128, 128), 64, 1, 81)


def test_attn_in_bf16_two_epochs_no_dx(b):
    _attn_in_case(b, "bf16", 200, 256, (256, 256), 16, 2, 82, with_dX=False)


def test_attn_in_fp32_generic_kernels(b):
    _attn_in_case(b, "f32", 50, 96, (96, 64, 64), 8, 1, 83)


def test_attn_in_7b_shape(b):
    # the 7B block's q, k, v at the metric's chunk size
    _attn_in_case(b, "bf16", 1024, 4096, (4096, 4096, 4096), 64, 1, 84)


def test_attn_in_argument_errors_launch_nothing(b):
    hosts = [inputs.make_linear(85, f"attnerr{i}", 64, 128, 128, 8, dtype="bf16") for i in range(2)]
    states = [make_state(h, "bf16") for h in hosts]
    lins = [b.linear_desc(h["W0"].cuda(), st["A"]["work"], st["B"]["work"], 2.0) for h, st in zip(hosts, states)]
    As = [b.param_desc(st["A"]["master"], st["A"]["m"], st["A"]["v"], st["A"]["grad"], st["A"]["work"]) for st in states]
    Bs = [b.param_desc(st["B"]["master"], st["B"]["m"], st["B"]["v"], st["B"]["grad"], st["B"]["work"]) for st in states]
    x = hosts[0]["x"].cuda()
    w = torch.ones(128, dtype=torch.bfloat16, device="cuda")
    xn = torch.full_like(x, float("nan"))
    dXn = torch.full_like(x, float("nan"))
    ys = [torch.empty((64, 128), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    dYs = [h["dY"].cuda() for h in hosts]
    short = b.alloc_workspace(2048)      # too small for the update: refused before the norm is enqueued
    with pytest.raises(b.TemploraError) as e:
        b.templora_update_attn_in(lins, As, Bs, x, w, 1e-5, dYs, xn, ys, dXn, None, 1, 1e-4, 0.9, 0.999, 1e-8, 0.0, 0, short)
    assert e.value.code == b.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert bool(torch.isnan(xn).all()), "the norm ran although the call was refused"
