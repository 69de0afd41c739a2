"""templora_update_mlp: the chunk update of a decoder block's MLP (gate, up -> SiLU gating -> down) in one call,
with the gating fused into the GEMM epilogues on the tensor-core path, against a composition of the oracle's
functions (linear_fwd / linear_bwd / swiglu_fwd / swiglu_bwd / adamw_step: no arithmetic of its own here)."""
import numpy as np
import pytest
import torch

from oracle import templora_oracle as orc
from paper_2401_11504_b200 import inputs
from parity_utils import (TOL, Guarded, assert_close, check_adam_steps, f64, hp32, ill_conditioned_mask, make_state)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2401_11504_b200 import build
    build.build_library()
    from paper_2401_11504_b200 import binding
    binding.templora_set_kernel_path(0)
    yield binding
    binding.templora_set_kernel_path(0)


def oracle_mlp(x, dY, W0, A0, B0, s, epochs, hp, bf16_work):
    """The MLP's chunk update composed from the oracle: W0, A0, B0 are lists (gate, up, down) of fp64 arrays.
    Returns the last epoch's tensors, the final state and the per-step gradient record."""
    A, B = [a.copy() for a in A0], [c.copy() for c in B0]
    mA, vA = [np.zeros_like(a) for a in A], [np.zeros_like(a) for a in A]
    mB, vB = [np.zeros_like(c) for c in B], [np.zeros_like(c) for c in B]
    log, out = [], {}
    for e in range(epochs):
        Aw = [orc.round_bf16(a) if bf16_work else a for a in A]
        Bw = [orc.round_bf16(c) if bf16_work else c for c in B]
        gate, _ = orc.linear_fwd(x, W0[0], Aw[0], Bw[0], s)
        up, _ = orc.linear_fwd(x, W0[1], Aw[1], Bw[1], s)
        h = orc.swiglu_fwd(gate, up)
        y, _ = orc.linear_fwd(h, W0[2], Aw[2], Bw[2], s)
        dh, dA_d, dB_d = orc.linear_bwd(h, dY, W0[2], Aw[2], Bw[2], s)
        dgate, dup = orc.swiglu_bwd(gate, up, dh)
        dXg, dA_g, dB_g = orc.linear_bwd(x, dgate, W0[0], Aw[0], Bw[0], s)
        dXu, dA_u, dB_u = orc.linear_bwd(x, dup, W0[1], Aw[1], Bw[1], s)
        dA, dB = [dA_g, dA_u, dA_d], [dB_g, dB_u, dB_d]
        out = dict(gate=gate, up=up, h=h, y=y, dX=dXg + dXu, dA=dA, dB=dB)
        for i in range(3):
            log.append((e + 1, i, dA[i].copy(), dB[i].copy()))
            A[i], mA[i], vA[i] = orc.adamw_step(A[i], dA[i], mA[i], vA[i], hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
                                                hp["weight_decay"], e + 1)
            B[i], mB[i], vB[i] = orc.adamw_step(B[i], dB[i], mB[i], vB[i], hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
                                                hp["weight_decay"], e + 1)
    out.update(A=A, B=B, mA=mA, mB=mB, vA=vA, vB=vB)
    return out, log


def _mlp_case(b, dtype, T, d, d_ff, ranks, epochs, hp, seed, with_dX=True, d_out=None):
    hp = hp32(hp)
    s = 2.0
    d_out = d_out or d
    shapes = [(d, d_ff, ranks[0]), (d, d_ff, ranks[1]), (d_ff, d_out, ranks[2])]
    hosts = [inputs.make_linear(seed, f"mlp{i}", T, di, do, r, dtype=dtype) for i, (di, do, r) in enumerate(shapes)]
    x_h, dY_h = hosts[0]["x"], hosts[2]["dY"]
    states = [make_state(hh, dtype) for hh in hosts]
    W0 = [hh["W0"].cuda() for hh in hosts]
    lins, As, Bs = [], [], []
    for w, st in zip(W0, states):
        a = st["A"]["work"] if dtype == "bf16" else st["A"]["master"]
        bb = st["B"]["work"] if dtype == "bf16" else st["B"]["master"]
        lins.append(b.linear_desc(w, a, bb, s))
        As.append(b.param_desc(st["A"]["master"], st["A"]["m"], st["A"]["v"], st["A"]["grad"], st["A"]["work"]))
        Bs.append(b.param_desc(st["B"]["master"], st["B"]["m"], st["B"]["v"], st["B"]["grad"], st["B"]["work"]))
    td = x_h.dtype
    guard = Guarded()
    gate, up, hbuf = (guard.empty((T, d_ff), td) for _ in range(3))
    y = guard.empty((T, d_out), td)
    dX = guard.empty((T, d), td) if with_dX else None
    ws = guard.workspace(b.templora_update_mlp_workspace_bytes(lins, T))
    x, dY = x_h.cuda(), dY_h.cuda()
    step = b.templora_update_mlp(lins, As, Bs, x, dY, gate, up, hbuf, y, dX, epochs, hp["lr"], hp["beta1"], hp["beta2"],
                                 hp["eps"], hp["weight_decay"], 0, ws)
    assert step == epochs
    assert b.templora_read_device_status(ws) == (0, 0)
    guard.check("after templora_update_mlp")

    ref, log = oracle_mlp(f64(x_h), f64(dY_h), [f64(hh["W0"]) for hh in hosts], [f64(hh["A"]) for hh in hosts],
                          [f64(hh["B"]) for hh in hosts], s, epochs, hp, dtype == "bf16")
    tol = TOL[dtype]
    errs = {}
    for name, got in (("gate", gate), ("up", up), ("h", hbuf), ("y", y)) + ((("dX", dX),) if with_dX else ()):
        errs[name] = assert_close(name, f64(got), ref[name], tol)
    for i, nm in enumerate(("gate", "up", "down")):
        st = states[i]
        errs[f"dA.{nm}"] = assert_close(f"dA.{nm}", f64(st["A"]["grad"]), ref["dA"][i], tol)
        errs[f"dB.{nm}"] = assert_close(f"dB.{nm}", f64(st["B"]["grad"]), ref["dB"][i], tol)
        for P in ("A", "B"):
            p0 = f64(hosts[i][P])
            got = f64(st[P]["master"])
            mask = ill_conditioned_mask(log, i, P, p0, hp, tol)
            check_adam_steps(f"{nm}.{P}", p0, got, ref[P][i], mask, tol, epochs, hp["lr"],
                             max_frac=0.03 if dtype == "bf16" else 1e-3)
            assert_close(f"m{P}.{nm}", f64(st[P]["m"]), ref["m" + P][i], tol)
            assert_close(f"v{P}.{nm}", f64(st[P]["v"]), ref["v" + P][i], 2 * tol)
            if epochs == 1:   # the optimizer's arithmetic, tightly: the oracle's step fed with the device's gradient
                g_dev = f64(st[P]["grad"])
                p1, _, _ = orc.adamw_step(p0, g_dev, 0 * p0, 0 * p0, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
                                          hp["weight_decay"], 1)
                tight = 1e-5 * np.abs(p1 - p0).max() + 2.0 ** -23 * np.abs(p1).max()
                assert np.abs((got - p0) - (p1 - p0)).max() <= tight
            if dtype == "bf16":
                assert np.array_equal(f64(st[P]["work"]), orc.round_bf16(got.astype(np.float32)))
    print("MLP worst relative errors:", {k: f"{v:.2e}" for k, v in errs.items()})


ADAM = dict(lr=2e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0)


@pytest.mark.parametrize("T,d,d_ff,r", [(200, 256, 704, 64), (300, 512, 1160, 16), (128, 256, 256, 128)])
def test_mlp_fused_gating_ragged_shapes(b, T, d, d_ff, r):
    # d_ff not a multiple of the 128-column tiles, T not a multiple of the 256-row tiles
    _mlp_case(b, "bf16", T, d, d_ff, (r, r, r), 1, ADAM, 61)


def test_mlp_two_epochs_and_no_input_gradient(b):
    _mlp_case(b, "bf16", 256, 256, 640, (64, 64, 64), 2, ADAM, 62)
    _mlp_case(b, "bf16", 256, 256, 640, (64, 64, 64), 1, ADAM, 63, with_dX=False)


def test_mlp_down_projects_to_another_width(b):
    _mlp_case(b, "bf16", 200, 256, 512, (64, 64, 32), 1, ADAM, 64, d_out=384)


def test_mlp_unfused_forms(b):
    # different ranks for gate and up: separate GEMMs and gating kernels on the tensor-core path
    _mlp_case(b, "bf16", 200, 256, 704, (64, 32, 64), 1, ADAM, 65)
    # single-CTA tiles (kernel path 2) and the generic kernels (path 1; fp32 too)
    for path in (2, 1):
        b.templora_set_kernel_path(path)
        try:
            _mlp_case(b, "bf16", 130, 128, 264, (16, 16, 16), 1, ADAM, 66 + path)
        finally:
            b.templora_set_kernel_path(0)
    _mlp_case(b, "f32", 70, 96, 80, (8, 8, 8), 2, dict(ADAM, weight_decay=0.01), 69)


def test_mlp_7b_shape_full(b):
    # the 7B block's MLP at the metric's chunk size: d = 4096, d_ff = 11008, T = 1024, rank 64
    _mlp_case(b, "bf16", 1024, 4096, 11008, (64, 64, 64), 1, dict(inputs.ADAMW), 70)


def test_mlp_rejects_mismatched_projections(b):
    W = lambda o, i: torch.zeros((o, i), dtype=torch.bfloat16, device="cuda")
    lins = [b.linear_desc(W(256, 128), W(16, 128), W(256, 16), 2.0), b.linear_desc(W(256, 128), W(16, 128), W(256, 16), 2.0),
            b.linear_desc(W(128, 192), W(16, 192), W(128, 16), 2.0)]     # down reads 192, the gating gives 256
    assert b.templora_update_mlp_workspace_bytes(lins, 64) == 0
