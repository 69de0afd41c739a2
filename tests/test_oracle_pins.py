"""Pins for the fp64 oracle: it is checked against things other than itself.

Brute-force scalar loops, a hand-worked integer example, algebraic identities
of the LoRA-augmented projection, exact finite differences, and closed forms of
AdamW.  The last test plants plausible mistakes in copies of the oracle and
requires that the pins catch each of them.
"""
import math

import numpy as np
import pytest
import torch

from conftest import load_golden
from oracle import templora_oracle as orc

RNG = np.random.default_rng(1234)


def rnd(*shape):
    return RNG.standard_normal(shape)


# ----------------------------------------------------------------- brute force
def brute_fwd(x, W0, A, B, s):
    T, d_in = x.shape
    d_out, r = B.shape
    y = [[0.0] * d_out for _ in range(T)]
    for t in range(T):
        u = [sum(x[t][k] * A[j][k] for k in range(d_in)) for j in range(r)]
        for o in range(d_out):
            base = sum(x[t][k] * W0[o][k] for k in range(d_in))
            low = sum(u[j] * B[o][j] for j in range(r))
            y[t][o] = base + s * low
    return np.array(y)


def brute_bwd(x, dY, W0, A, B, s):
    T, d_in = x.shape
    d_out, r = B.shape
    dX = np.zeros((T, d_in)); dA = np.zeros((r, d_in)); dB = np.zeros((d_out, r))
    for t in range(T):
        u = [sum(x[t][k] * A[j][k] for k in range(d_in)) for j in range(r)]
        v = [sum(dY[t][o] * B[o][j] for o in range(d_out)) for j in range(r)]
        for k in range(d_in):
            dX[t][k] = sum(dY[t][o] * W0[o][k] for o in range(d_out)) + s * sum(v[j] * A[j][k] for j in range(r))
        for o in range(d_out):
            for j in range(r):
                dB[o][j] += s * dY[t][o] * u[j]
        for j in range(r):
            for k in range(d_in):
                dA[j][k] += s * v[j] * x[t][k]
    return dX, dA, dB


SHAPES = [(5, 7, 6, 3), (1, 4, 9, 2), (9, 3, 2, 5)]


@pytest.mark.parametrize("T,d_in,d_out,r", SHAPES)
def test_fwd_bwd_match_scalar_loops(T, d_in, d_out, r):
    x, W0, A, B, dY = rnd(T, d_in), rnd(d_out, d_in), rnd(r, d_in), rnd(d_out, r), rnd(T, d_out)
    s = 1.75
    y, U = orc.linear_fwd(x, W0, A, B, s)
    np.testing.assert_allclose(y, brute_fwd(x, W0, A, B, s), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(U, x @ A.T, rtol=1e-13, atol=1e-13)
    dX, dA, dB = orc.linear_bwd(x, dY, W0, A, B, s)
    bX, bA, bB = brute_bwd(x, dY, W0, A, B, s)
    np.testing.assert_allclose(dX, bX, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dA, bA, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dB, bB, rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------ worked example
def test_hand_worked_integer_case():
    g = load_golden("lora_integer_case.txt")
    s = float(g["s"][0, 0])
    y, U = orc.linear_fwd(g["x"], g["W0"], g["A"], g["B"], s)
    assert np.array_equal(y, g["y"]) and np.array_equal(U, g["U"])
    dX, dA, dB = orc.linear_bwd(g["x"], g["dY"], g["W0"], g["A"], g["B"], s)
    assert np.array_equal(dX, g["dX"]) and np.array_equal(dA, g["dA"]) and np.array_equal(dB, g["dB"])
    assert np.array_equal(orc.decode_fwd(g["x"], g["W0"], g["A"], g["B"], s), g["y"])


# ----------------------------------------------------------------- identities
def test_zero_B_reduces_to_base_linear_exactly():
    T, d_in, d_out, r = 6, 11, 5, 4
    x, W0, A, dY = rnd(T, d_in), rnd(d_out, d_in), rnd(r, d_in), rnd(T, d_out)
    B = np.zeros((d_out, r))
    y, _ = orc.linear_fwd(x, W0, A, B, 2.0)
    assert np.array_equal(y, x @ W0.T)          # bit for bit
    dX, dA, dB = orc.linear_bwd(x, dY, W0, A, B, 2.0)
    assert np.array_equal(dX, dY @ W0)
    assert not dA.any()                         # no gradient reaches A through B = 0
    assert np.abs(dB).max() > 0
    # A = 0 kills dB and the low-rank part of dX
    dX2, dA2, dB2 = orc.linear_bwd(x, dY, W0, np.zeros_like(A), rnd(d_out, r), 2.0)
    assert not dB2.any() and np.array_equal(dX2, dY @ W0)


def test_merged_weight_identity():
    T, d_in, d_out, r, s = 8, 13, 10, 4, 2.0
    x, W0, A, B, dY = rnd(T, d_in), rnd(d_out, d_in), rnd(r, d_in), rnd(d_out, r), rnd(T, d_out)
    Wm = W0 + s * (B @ A)
    y, _ = orc.linear_fwd(x, W0, A, B, s)
    dX, _, _ = orc.linear_bwd(x, dY, W0, A, B, s)
    np.testing.assert_allclose(y, x @ Wm.T, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dX, dY @ Wm, rtol=1e-12, atol=1e-12)


def test_linear_in_s():
    T, d_in, d_out, r = 4, 6, 5, 3
    x, W0, A, B = rnd(T, d_in), rnd(d_out, d_in), rnd(r, d_in), rnd(d_out, r)
    y0, _ = orc.linear_fwd(x, W0, A, B, 0.0)
    y1, _ = orc.linear_fwd(x, W0, A, B, 1.0)
    y3, _ = orc.linear_fwd(x, W0, A, B, 3.0)
    np.testing.assert_allclose(y3 - y0, 3.0 * (y1 - y0), rtol=1e-12, atol=1e-12)


def _loss(x, W0, A, B, s, dY):
    y, _ = orc.linear_fwd(x, W0, A, B, s)
    return float((dY * y).sum())


def test_gradients_match_exact_finite_differences():
    # L = sum(dY * y) is linear in each of x, A, B taken alone, so a central
    # difference with ANY step is exact up to rounding.
    T, d_in, d_out, r, s, h = 5, 7, 6, 3, 2.0, 0.5
    x, W0, A, B, dY = rnd(T, d_in), rnd(d_out, d_in), rnd(r, d_in), rnd(d_out, r), rnd(T, d_out)
    dX, dA, dB = orc.linear_bwd(x, dY, W0, A, B, s)

    def fd(arr, which):
        g = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            plus, minus = arr.copy(), arr.copy()
            plus[idx] += h; minus[idx] -= h
            args_p = dict(x=x, A=A, B=B); args_m = dict(x=x, A=A, B=B)
            args_p[which] = plus; args_m[which] = minus
            g[idx] = (_loss(args_p["x"], W0, args_p["A"], args_p["B"], s, dY)
                      - _loss(args_m["x"], W0, args_m["A"], args_m["B"], s, dY)) / (2 * h)
        return g

    for got, ref in ((dX, fd(x, "x")), (dA, fd(A, "A")), (dB, fd(B, "B"))):
        assert np.abs(got - ref).max() <= 1e-9 * max(1.0, np.abs(ref).max())


def test_dA_dB_additive_over_row_partitions():
    T, d_in, d_out, r, s = 11, 6, 7, 3, 2.0
    x, W0, A, B, dY = rnd(T, d_in), rnd(d_out, d_in), rnd(r, d_in), rnd(d_out, r), rnd(T, d_out)
    dX, dA, dB = orc.linear_bwd(x, dY, W0, A, B, s)
    cut = 4
    dX1, dA1, dB1 = orc.linear_bwd(x[:cut], dY[:cut], W0, A, B, s)
    dX2, dA2, dB2 = orc.linear_bwd(x[cut:], dY[cut:], W0, A, B, s)
    np.testing.assert_allclose(dA, dA1 + dA2, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dB, dB1 + dB2, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dX, np.vstack([dX1, dX2]), rtol=1e-13, atol=1e-13)


def test_decode_equals_rows_of_chunk_forward():
    d_in, d_out, r, s = 24, 17, 4, 2.0
    W0, A, B = rnd(d_out, d_in), rnd(r, d_in), rnd(d_out, r)
    for n in (1, 4, 16):
        x = rnd(n, d_in)
        y, _ = orc.linear_fwd(x, W0, A, B, s)
        np.testing.assert_allclose(orc.decode_fwd(x, W0, A, B, s), y, rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------------- AdamW
def test_adamw_hand_worked_first_step():
    g = {k: float(v[0, 0]) for k, v in load_golden("adamw_first_step.txt").items()}
    p, m, v = orc.adamw_step([g["p0"]], [g["g"]], [0.0], [0.0], g["lr"], g["beta1"], g["beta2"],
                             g["eps"], g["wd"], 1)
    assert abs(p[0] - g["p1"]) < 1e-15
    assert abs(m[0] - g["m1"]) < 1e-16 and abs(v[0] - g["v1"]) < 1e-18


def test_adamw_first_step_closed_form():
    p0, g = rnd(50), rnd(50)
    lr, b1, b2, eps, wd = 3e-3, 0.9, 0.999, 1e-8, 0.05
    p, m, v = orc.adamw_step(p0, g, np.zeros(50), np.zeros(50), lr, b1, b2, eps, wd, 1)
    np.testing.assert_allclose(p, p0 * (1 - lr * wd) - lr * g / (np.abs(g) + eps), rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(m, (1 - b1) * g, rtol=1e-13)
    np.testing.assert_allclose(v, (1 - b2) * g * g, rtol=1e-12)


def test_adamw_zero_gradient_leaves_parameters():
    p0 = rnd(20)
    p, m, v = orc.adamw_step(p0, np.zeros(20), np.zeros(20), np.zeros(20), 5e-5, 0.9, 0.999, 1e-8, 0.0, 1)
    assert np.array_equal(p, p0) and not m.any() and not v.any()


def test_adamw_constant_gradient_trajectory():
    # with a constant gradient m_hat = g and v_hat = g^2 at every step, so
    # p_k = p0 - k lr g / (|g| + eps): pins the bias correction for t > 1
    p0, g = rnd(30), rnd(30)
    lr, eps = 1e-3, 1e-8
    p, m, v = p0.copy(), np.zeros(30), np.zeros(30)
    for t in range(1, 8):
        p, m, v = orc.adamw_step(p, g, m, v, lr, 0.9, 0.999, eps, 0.0, t)
        np.testing.assert_allclose(p, p0 - t * lr * g / (np.abs(g) + eps), rtol=1e-10, atol=1e-13)


def test_adamw_sign_antisymmetry_and_torch():
    p0, g = rnd(40), rnd(40)
    a = orc.adamw_step(p0, g, np.zeros(40), np.zeros(40), 1e-3, 0.9, 0.999, 1e-8, 0.0, 1)[0]
    b = orc.adamw_step(-p0, -g, np.zeros(40), np.zeros(40), 1e-3, 0.9, 0.999, 1e-8, 0.0, 1)[0]
    np.testing.assert_allclose(a, -b, rtol=1e-14)
    # an independent implementation: torch.optim.AdamW in float64, several steps, wd != 0
    tp = torch.tensor(p0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.AdamW([tp], lr=2e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.1)
    p, m, v = p0.copy(), np.zeros(40), np.zeros(40)
    for t in range(1, 5):
        gt = g * t
        tp.grad = torch.tensor(gt, dtype=torch.float64)
        opt.step()
        p, m, v = orc.adamw_step(p, gt, m, v, 2e-3, 0.9, 0.999, 1e-8, 0.1, t)
        np.testing.assert_allclose(p, tp.detach().numpy(), rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------------- rounding
def test_round_bf16_matches_torch_cast():
    vals = np.concatenate([rnd(5000).astype(np.float32) * np.float32(10.0 ** RNG.integers(-6, 6)),
                           np.array([0.0, -0.0, 1.0, 1.00390625, 1.0078125, 3.0e38, 1e-40, -1e-40,
                                     np.inf, -np.inf], dtype=np.float32)])
    # exact ties: mantissa bit pattern xxxx 1000 0000 0000 0000
    ties = (np.arange(256, dtype=np.uint32) << np.uint32(16) | np.uint32(0x3F800000) | np.uint32(0x8000)).view(np.float32)
    vals = np.concatenate([vals, ties])
    ref = torch.from_numpy(vals).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(orc.round_bf16(vals), ref)


# --------------------------------------------------------------- update_block
def _mk_proj(T, d_in, d_out, r, s):
    return dict(x=rnd(T, d_in), dY=rnd(T, d_out), W0=rnd(d_out, d_in) / math.sqrt(d_in), s=s,
                A_master=rnd(r, d_in) * 0.1, B_master=rnd(d_out, r) * 0.1)


def test_update_block_single_epoch_is_the_composition():
    projs = [_mk_proj(6, 8, 5, 2, 2.0), _mk_proj(6, 5, 9, 2, 2.0)]
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    st, step = orc.update_block(projs, 1, **hp)
    assert step == 1
    for p, q in zip(projs, st):
        dX, dA, dB = orc.linear_bwd(p["x"], p["dY"], p["W0"], p["A_master"], p["B_master"], p["s"])
        A1, mA, vA = orc.adamw_step(p["A_master"], dA, 0 * dA, 0 * dA, t=1, **hp)
        B1, mB, vB = orc.adamw_step(p["B_master"], dB, 0 * dB, 0 * dB, t=1, **hp)
        assert np.array_equal(q["A_master"], A1) and np.array_equal(q["B_master"], B1)
        assert np.array_equal(q["dX"], dX) and np.array_equal(q["mA"], mA) and np.array_equal(q["vB"], vB)


def test_update_block_two_epochs_and_zero_lr():
    projs = [_mk_proj(7, 6, 4, 3, 2.0)]
    hp = dict(lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0)
    st2, step = orc.update_block(projs, 2, **hp)
    assert step == 2
    # by hand: epoch 2 starts from epoch 1's result, moments and step carried over
    st1, _ = orc.update_block(projs, 1, **hp)
    p2 = [dict(projs[0], A_master=st1[0]["A_master"], B_master=st1[0]["B_master"],
               mA=st1[0]["mA"], vA=st1[0]["vA"], mB=st1[0]["mB"], vB=st1[0]["vB"])]
    st12, step12 = orc.update_block(p2, 1, step0=1, **hp)
    assert step12 == 2
    assert np.array_equal(st2[0]["A_master"], st12[0]["A_master"])
    assert np.array_equal(st2[0]["B_master"], st12[0]["B_master"])
    # the second epoch really sees the updated module
    assert np.abs(st2[0]["y"] - st1[0]["y"]).max() > 0
    # lr = 0: nothing moves, epoch 2 repeats epoch 1
    hp0 = dict(hp, lr=0.0)
    a, _ = orc.update_block(projs, 1, **hp0)
    b, _ = orc.update_block(projs, 2, **hp0)
    assert np.array_equal(a[0]["y"], b[0]["y"]) and np.array_equal(a[0]["dA"], b[0]["dA"])
    assert np.array_equal(b[0]["A_master"], projs[0]["A_master"])


def test_update_block_bf16_working_copy():
    projs = [_mk_proj(4, 8, 8, 2, 2.0)]
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0)
    st, _ = orc.update_block(projs, 1, bf16_work=True, **hp)
    Aw, Bw = orc.round_bf16(projs[0]["A_master"]), orc.round_bf16(projs[0]["B_master"])
    y, _ = orc.linear_fwd(projs[0]["x"], projs[0]["W0"], Aw, Bw, 2.0)
    assert np.array_equal(st[0]["y"], y)
    # the optimizer moves the un-rounded master
    _, dA, _ = orc.linear_bwd(projs[0]["x"], projs[0]["dY"], projs[0]["W0"], Aw, Bw, 2.0)
    A1, _, _ = orc.adamw_step(projs[0]["A_master"], dA, 0 * dA, 0 * dA, t=1, **hp)
    assert np.array_equal(st[0]["A_master"], A1)


# -------------------------------------------- the pins catch planted mistakes
def _pins_pass(fwd, bwd):
    g = load_golden("lora_integer_case.txt")
    s = float(g["s"][0, 0])
    try:
        y, _ = fwd(g["x"], g["W0"], g["A"], g["B"], s)
        dX, dA, dB = bwd(g["x"], g["dY"], g["W0"], g["A"], g["B"], s)
        ok = all(np.array_equal(a, b) for a, b in ((y, g["y"]), (dX, g["dX"]), (dA, g["dA"]), (dB, g["dB"])))
        T, d_in, d_out, r = 5, 7, 6, 3
        rs = np.random.default_rng(7)
        x, W0, A, B, dY = (rs.standard_normal(sh) for sh in ((T, d_in), (d_out, d_in), (r, d_in), (d_out, r), (T, d_out)))
        y, _ = fwd(x, W0, A, B, 1.5)
        dX, dA, dB = bwd(x, dY, W0, A, B, 1.5)
        bX, bA, bB = brute_bwd(x, dY, W0, A, B, 1.5)
        ok = ok and np.allclose(y, brute_fwd(x, W0, A, B, 1.5), rtol=1e-11, atol=1e-11)
        ok = ok and np.allclose(dX, bX, rtol=1e-11, atol=1e-11) and np.allclose(dA, bA, rtol=1e-11, atol=1e-11)
        ok = ok and np.allclose(dB, bB, rtol=1e-11, atol=1e-11)
        return bool(ok)
    except Exception:
        return False


def test_pins_catch_planted_mistakes():
    assert _pins_pass(orc.linear_fwd, orc.linear_bwd)
    f, b = orc.linear_fwd, orc.linear_bwd
    wrong_fwd = [
        lambda x, W0, A, B, s: (x @ W0.T + (x @ A.T) @ B.T, x @ A.T),               # dropped s
        lambda x, W0, A, B, s: (x @ W0.T - s * (x @ A.T) @ B.T, x @ A.T),           # wrong sign
        lambda x, W0, A, B, s: (x @ W0.T + s * s * (x @ A.T) @ B.T, x @ A.T),       # s applied twice
        lambda x, W0, A, B, s: (x @ W0.T, x @ A.T),                                  # dropped term
    ]
    for wf in wrong_fwd:
        assert not _pins_pass(wf, b)

    def bwd_variant(kind):
        def fn(x, dY, W0, A, B, s):
            U, V = x @ A.T, dY @ B
            dX = dY @ W0 + s * (V @ A)
            dB = s * (dY.T @ U)
            dA = s * (V.T @ x)
            if kind == "dX_no_lora": dX = dY @ W0
            if kind == "dB_no_s": dB = dY.T @ U
            if kind == "dA_uses_U": dA = s * (U.T @ x)
            if kind == "dB_uses_V": dB = s * (dY.T @ V)
            if kind == "dA_mean": dA = dA / x.shape[0]
            return dX, dA, dB
        return fn
    for kind in ("dX_no_lora", "dB_no_s", "dA_uses_U", "dB_uses_V", "dA_mean"):
        assert not _pins_pass(f, bwd_variant(kind))


def test_update_block_batches_are_sequential_updates_on_row_slices():
    # chunk 10, batch 4, 2 epochs: 2 * ceil(10 / 4) = 6 optimizer steps (the cost table's count of
    # training steps); by hand: one single-batch update per row slice, state carried along
    projs = [_mk_proj(10, 6, 5, 2, 2.0), _mk_proj(10, 5, 7, 2, 2.0)]
    hp = dict(lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    st, step = orc.update_block(projs, 2, batch=4, **hp)
    assert step == 6
    cur = [dict(p) for p in projs]
    k = 0
    for _ in range(2):
        for r0, r1 in ((0, 4), (4, 8), (8, 10)):
            sl = [dict(c, x=c["x"][r0:r1], dY=c["dY"][r0:r1]) for c in cur]
            out, k = orc.update_block(sl, 1, step0=k, **hp)
            for c, o, full in zip(cur, out, st):
                for key in ("A_master", "B_master", "mA", "vA", "mB", "vB"):
                    c[key] = o[key]
                last = o
    assert k == 6
    for c, full in zip(cur, st):
        assert np.array_equal(c["A_master"], full["A_master"]) and np.array_equal(c["vB"], full["vB"])
    # batch >= T is the unbatched update, bit for bit
    a, _ = orc.update_block(projs, 2, **hp)
    b, _ = orc.update_block(projs, 2, batch=10, **hp)
    c, _ = orc.update_block(projs, 2, batch=64, **hp)
    for u, v, w in zip(a, b, c):
        assert np.array_equal(u["A_master"], v["A_master"]) and np.array_equal(u["y"], w["y"])
    # rows of y come from the slice's own parameter version: the first slice of the last epoch
    # was computed before the last two steps, so it differs from an unbatched pass with final weights
    assert st[0]["y"].shape == (10, 5)


# ------------------------------------------------------------------- dropout
def test_philox4x32_10_known_answers():
    # known-answer vectors published with the generator (Random123 distribution, kat_vectors)
    kat = [
        ((0, 0, 0, 0), (0, 0), (0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8)),
        ((0xffffffff,) * 4, (0xffffffff, 0xffffffff), (0x408f276d, 0x41c83b0e, 0xa20bc7c6, 0x6d5451fd)),
        ((0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344), (0xa4093822, 0x299f31d0),
         (0xd16cfe09, 0x94fdcceb, 0x5001e420, 0x24126ea1)),
    ]
    for ctr, key, want in kat:
        got = orc.philox4x32_10(np.array([ctr], dtype=np.uint32), key)[0]
        assert tuple(int(v) for v in got) == want


def test_dropout_keep_statistics_and_determinism():
    k1 = orc.dropout_keep(1234, 7, 300, 512, 0.05)
    assert k1.shape == (300, 512) and set(np.unique(k1)) <= {0, 1}
    assert abs(k1.mean() - 0.95) < 0.005                      # 153600 draws: sigma = 5.6e-4
    assert np.array_equal(k1, orc.dropout_keep(1234, 7, 300, 512, 0.05))
    assert not np.array_equal(k1, orc.dropout_keep(1234, 8, 300, 512, 0.05))     # next step, new mask
    assert not np.array_equal(k1, orc.dropout_keep(1235, 7, 300, 512, 0.05))
    assert orc.dropout_keep(1, 0, 8, 8, 0.0).all()
    # a larger p only drops more: same draws, higher threshold
    k5 = orc.dropout_keep(1234, 7, 300, 512, 0.5)
    assert abs(k5.mean() - 0.5) < 0.01 and not (k5 & ~k1).any()
    # a row slice of a longer chunk is NOT the same mask (the element index depends on the slice shape)
    assert orc.dropout_keep(9, 0, 4, 16, 0.3).shape == (4, 16)


# A scalar restatement of the generator and of the mask rule, in plain Python integers, sharing nothing
# with the oracle's vectorised code.  The generator is checked against its published vectors below
# before it is used as a yardstick.
_KAT = [
    ((0, 0, 0, 0), (0, 0), (0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8)),
    ((0xffffffff,) * 4, (0xffffffff, 0xffffffff), (0x408f276d, 0x41c83b0e, 0xa20bc7c6, 0x6d5451fd)),
    ((0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344), (0xa4093822, 0x299f31d0),
     (0xd16cfe09, 0x94fdcceb, 0x5001e420, 0x24126ea1)),
]


def _philox_scalar(ctr, key):
    c0, c1, c2, c3 = ctr
    k0, k1 = key
    for _ in range(10):
        lo0, hi0 = (0xD2511F53 * c0) & 0xFFFFFFFF, (0xD2511F53 * c0) >> 32
        lo1, hi1 = (0xCD9E8D57 * c2) & 0xFFFFFFFF, (0xCD9E8D57 * c2) >> 32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        k0, k1 = (k0 + 0x9E3779B9) & 0xFFFFFFFF, (k1 + 0xBB67AE85) & 0xFFFFFFFF
    return (c0, c1, c2, c3)


def _keep_by_rule(seed, offset, T, d_in, p):
    """The mask rule of the library's header, element by element: element e = t*d_in + k takes word e % 4 of
    the block whose counter is (lo(e/4), hi(e/4), lo(offset), hi(offset)) under key (lo(seed), hi(seed));
    dropped iff that word < floor(p * 2^32)."""
    thr = int(math.floor(p * 4294967296.0))
    lo, hi = (lambda v: v & 0xFFFFFFFF), (lambda v: (v >> 32) & 0xFFFFFFFF)
    keep = np.zeros((T, d_in), dtype=np.uint8)
    for t in range(T):
        for k in range(d_in):
            e = t * d_in + k
            word = _philox_scalar((lo(e // 4), hi(e // 4), lo(offset), hi(offset)), (lo(seed), hi(seed)))[e % 4]
            keep[t, k] = 0 if word < thr else 1
    return keep


def _dropout_layout_pins_pass(keep_fn):
    try:
        # (1) first published vector: counter (0,0,0,0), key (0,0) -> 6627e8d5 e169c58d bc57ac4c 9b00dbd8.
        #     seed 0, offset 0, one row of four elements, p = 0.5 (threshold 0x80000000): only the first
        #     word is below the threshold, so element 0 is dropped and elements 1..3 are kept.
        ok = np.array_equal(keep_fn(0, 0, 1, 4, 0.5), np.array([[0, 1, 1, 1]], dtype=np.uint8))
        #     same draws against p = 0.75 (0xC0000000): 66.. 9b.. bc.. are below, e1.. is not.
        ok = ok and np.array_equal(keep_fn(0, 0, 1, 4, 0.75), np.array([[0, 1, 0, 0]], dtype=np.uint8))
        # (2) a 64-bit offset and a 64-bit seed whose low and high words differ, rows of 6 elements so that
        #     rows 1 and 2 start in the middle of a block (e = 6 -> block 1 word 2; e = 12 -> block 3 word 0),
        #     and 18 elements = four full blocks and a half
        seed, offset = 0x0123456789ABCDEF, 0x00000002_00000005
        for p in (0.5, 0.3):
            ok = ok and np.array_equal(keep_fn(seed, offset, 3, 6, p), _keep_by_rule(seed, offset, 3, 6, p))
        # (3) the step offset enters the counter, not the key: offset 1 with seed 0 is a different block
        #     from offset 0 with seed 1
        ok = ok and np.array_equal(keep_fn(0, 1, 2, 8, 0.5), _keep_by_rule(0, 1, 2, 8, 0.5))
        ok = ok and np.array_equal(keep_fn(1, 0, 2, 8, 0.5), _keep_by_rule(1, 0, 2, 8, 0.5))
        return bool(ok)
    except Exception:
        return False


def test_dropout_keep_layout_by_hand_and_by_scalar_rule():
    for ctr, key, want in _KAT:                    # the yardstick itself against the published vectors
        assert _philox_scalar(ctr, key) == want
    # the scalar rule reproduces the hand case too (so the yardstick's word order is the header's)
    assert np.array_equal(_keep_by_rule(0, 0, 1, 4, 0.5), [[0, 1, 1, 1]])
    assert _dropout_layout_pins_pass(orc.dropout_keep)
    # the cases of (2) are not degenerate: both values occur, and the 64-bit halves matter
    m = _keep_by_rule(0x0123456789ABCDEF, 0x00000002_00000005, 3, 6, 0.5)
    assert 0 < m.sum() < m.size
    assert not np.array_equal(m, _keep_by_rule(0x0123456789ABCDEF, 0x00000005_00000002, 3, 6, 0.5))
    assert not np.array_equal(m, _keep_by_rule(0x89ABCDEF01234567, 0x00000002_00000005, 3, 6, 0.5))


def test_dropout_layout_pins_catch_planted_mistakes():
    """Copies of the oracle's mask routine with one layout mistake each must fail the pins above."""
    def variant(kind):
        def fn(seed, offset, T, d_in, p):
            seed, offset = int(seed), int(offset)
            n = T * d_in
            lo, hi = (lambda v: v & 0xFFFFFFFF), (lambda v: (v >> 32) & 0xFFFFFFFF)
            key = (lo(seed), hi(seed))
            if kind == "key_halves_swapped": key = (hi(seed), lo(seed))
            thr = min(orc.dropout_threshold(p), 0xFFFFFFFF)
            out = np.zeros(n, dtype=np.uint8)
            for e in range(n):
                blk, word = e // 4, e % 4
                if kind == "rows_start_new_blocks":
                    t, k = divmod(e, d_in)
                    blk, word = t * ((d_in + 3) // 4) + k // 4, k % 4
                ctr = [lo(blk), hi(blk), lo(offset), hi(offset)]
                if kind == "offset_halves_swapped": ctr = [lo(blk), hi(blk), hi(offset), lo(offset)]
                if kind == "offset_in_words_0_1": ctr = [lo(offset), hi(offset), lo(blk), hi(blk)]
                if kind == "offset_added_to_index": ctr = [lo(blk + offset), hi(blk + offset), 0, 0]
                if kind == "offset_in_key": ctr, key = [lo(blk), hi(blk), 0, 0], (lo(seed + offset), hi(seed + offset))
                if kind == "words_reversed": word = 3 - word
                if kind == "one_block_per_element": ctr, word = [lo(e), hi(e), lo(offset), hi(offset)], 0
                draw = int(orc.philox4x32_10(np.array([ctr], dtype=np.uint32), key)[0][word])
                out[e] = (draw >= thr) if kind != "keeps_below_threshold" else (draw < thr)
            return out.reshape(T, d_in)
        return fn
    assert _dropout_layout_pins_pass(variant("none"))    # the copy without a mistake passes
    for kind in ("key_halves_swapped", "rows_start_new_blocks", "offset_halves_swapped", "offset_in_words_0_1",
                 "offset_added_to_index", "offset_in_key", "words_reversed", "one_block_per_element",
                 "keeps_below_threshold"):
        assert not _dropout_layout_pins_pass(variant(kind)), kind


def test_dropout_forward_backward_against_loops_and_differences():
    T, d_in, d_out, r, s, p = 5, 8, 6, 3, 2.0, 0.25
    x, W0, A, B, dY = rnd(T, d_in), rnd(d_out, d_in), rnd(r, d_in), rnd(d_out, r), rnd(T, d_out)
    keep = orc.dropout_keep(77, 3, T, d_in, p)
    assert 0 < keep.sum() < keep.size
    y, U = orc.linear_fwd(x, W0, A, B, s, keep, p)
    # scalar loops
    for t in range(T):
        u = [sum(x[t][k] * keep[t][k] / (1 - p) * A[j][k] for k in range(d_in)) for j in range(r)]
        for o in range(d_out):
            want = sum(x[t][k] * W0[o][k] for k in range(d_in)) + s * sum(u[j] * B[o][j] for j in range(r))
            assert abs(y[t][o] - want) < 1e-12
    # the loss sum(dY*y) stays linear in each of x, A, B with the mask held fixed: exact differences
    dX, dA, dB = orc.linear_bwd(x, dY, W0, A, B, s, keep, p)
    loss = lambda xx, AA, BB: float((dY * orc.linear_fwd(xx, W0, AA, BB, s, keep, p)[0]).sum())
    h = 0.5
    for arr, grad, which in ((x, dX, 0), (A, dA, 1), (B, dB, 2)):
        fd = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            plus, minus = arr.copy(), arr.copy()
            plus[idx] += h; minus[idx] -= h
            args_p, args_m = [x, A, B], [x, A, B]
            args_p[which], args_m[which] = plus, minus
            fd[idx] = (loss(*args_p) - loss(*args_m)) / (2 * h)
        assert np.abs(grad - fd).max() <= 1e-9 * max(1.0, np.abs(fd).max())
    # p = 0 / no mask is the plain projection, bit for bit; an all-ones mask with p = 0 too
    y0, _ = orc.linear_fwd(x, W0, A, B, s)
    y1, _ = orc.linear_fwd(x, W0, A, B, s, np.ones_like(keep), 0.0)
    assert np.array_equal(y0, y1)
    # dropped inputs get no gradient through the LoRA branch
    base = dY @ W0
    assert np.allclose((dX - base)[keep == 0], 0.0)


def test_update_block_with_dropout_draws_a_mask_per_step():
    projs = [dict(_mk_proj(8, 8, 6, 2, 2.0), dropout_seed=5), dict(_mk_proj(8, 6, 8, 2, 2.0), dropout_seed=6)]
    hp = dict(lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0)
    st, step = orc.update_block(projs, 2, dropout_p=0.5, batch=4, **hp)
    assert step == 4
    # by hand for the first step of projection 0: rows 0..3, offset 0 + 0 steps taken
    keep = orc.dropout_keep(5, 0, 4, 8, 0.5)
    p = projs[0]
    _, dA, dB = orc.linear_bwd(p["x"][:4], p["dY"][:4], p["W0"], p["A_master"], p["B_master"], 2.0, keep, 0.5)
    A1, _, _ = orc.adamw_step(p["A_master"], dA, 0 * dA, 0 * dA, t=1, **hp)
    one, _ = orc.update_block([dict(p, x=p["x"][:4], dY=p["dY"][:4])], 1, dropout_p=0.5, **hp)
    assert np.array_equal(one[0]["A_master"], A1)
    # and dropout changes the result
    plain, _ = orc.update_block(projs, 2, batch=4, **hp)
    assert np.abs(plain[0]["A_master"] - st[0]["A_master"]).max() > 0


# ------------------------------------------------------------------ learning-rate warm-up
def test_lr_warmup_closed_forms():
    # linear from lr/w at step 1 to lr at step w, constant after; w <= 0 switches it off
    lr, w = 5e-5, 8
    vals = [orc.lr_at_step(lr, k, w) for k in range(1, 13)]
    assert vals[0] == pytest.approx(lr / w, rel=1e-15)
    assert vals[w - 1] == lr and all(v == lr for v in vals[w:])
    diffs = np.diff(vals[:w])
    assert np.allclose(diffs, lr / w, rtol=1e-12)
    assert orc.lr_at_step(lr, 1, 0) == lr and orc.lr_at_step(lr, 3, -1) == lr


def test_update_block_warmup_equals_steps_composed_by_hand():
    # one call over 2 epochs x 2 batches with warm-up = four single-batch calls, each with its own rate
    # and the running step count; pins which step number each rate belongs to
    rng = np.random.default_rng(5)
    T, d_in, d_out, r = 8, 6, 5, 2
    p0 = dict(x=rng.normal(size=(T, d_in)), dY=rng.normal(size=(T, d_out)), W0=rng.normal(size=(d_out, d_in)), s=1.5,
              A_master=rng.normal(size=(r, d_in)), B_master=rng.normal(size=(d_out, r)))
    hp = dict(lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)
    ref, step = orc.update_block([p0], 2, **hp, batch=4, warmup_steps=3)
    assert step == 4
    cur, k = dict(p0), 0
    for _ in range(2):
        for rows in (slice(0, 4), slice(4, 8)):
            q = dict(cur, x=p0["x"][rows], dY=p0["dY"][rows])
            hp_k = dict(hp, lr=hp["lr"] * min(1.0, (k + 1) / 3.0))
            out, k = orc.update_block([q], 1, **hp_k, step0=k)
            cur.update({n: out[0][n] for n in ("A_master", "B_master", "mA", "vA", "mB", "vB")})
    for n in ("A_master", "B_master", "mA", "vA", "mB", "vB"):
        assert np.allclose(ref[0][n], cur[n], rtol=1e-13, atol=1e-15), n


# ------------------------------------------------------------------ shared-input projections
def test_summed_input_gradient_matches_finite_differences():
    # q, k, v read the same x: with L = sum_i <dY_i, y_i(x)>, dL/dx is the sum of the three input
    # gradients; L is linear in x, so central differences are exact up to rounding
    rng = np.random.default_rng(11)
    T, d_in, r = 4, 6, 2
    x = rng.normal(size=(T, d_in))
    projs = []
    for i, d_out in enumerate((5, 3, 4)):
        projs.append(dict(x=x, dY=rng.normal(size=(T, d_out)), W0=rng.normal(size=(d_out, d_in)), s=0.7 + i,
                          A_master=rng.normal(size=(r, d_in)), B_master=rng.normal(size=(d_out, r)),
                          dX_to=None if i == 0 else 0))
    st, _ = orc.update_block(projs, 1, 0.0, 0.9, 0.999, 1e-8, 0.0)
    assert st[1]["dX"] is st[0]["dX"] and st[2]["dX"] is st[0]["dX"]

    def loss(xx):
        return sum(np.sum(p["dY"] * orc.linear_fwd(xx, p["W0"], p["A_master"], p["B_master"], p["s"])[0]) for p in projs)
    h = 1e-3
    fd = np.zeros_like(x)
    for t in range(T):
        for k in range(d_in):
            e = np.zeros_like(x); e[t, k] = h
            fd[t, k] = (loss(x + e) - loss(x - e)) / (2 * h)
    assert np.allclose(st[0]["dX"], fd, rtol=1e-9, atol=1e-9)
    # and it is not any single projection's gradient
    alone, _ = orc.update_block([dict(projs[0], dX_to=None)], 1, 0.0, 0.9, 0.999, 1e-8, 0.0)
    assert not np.allclose(alone[0]["dX"], fd)


# ------------------------------------------------------------------ SiLU gating and RMSNorm
def _fd(f, x, h=1e-6):
    g = np.zeros_like(x)
    it = np.nditer(x, flags=["multi_index"])
    for _ in it:
        e = np.zeros_like(x); e[it.multi_index] = h
        g[it.multi_index] = (f(x + e) - f(x - e)) / (2 * h)
    return g


def test_swiglu_values_and_gradients():
    # SiLU(0) = 0, SiLU'(0) = 1/2, SiLU(g) -> g for large g, -> 0 for very negative g
    assert orc.swiglu_fwd(np.array([[0.0]]), np.array([[3.0]]))[0, 0] == 0.0
    dg, du = orc.swiglu_bwd(np.array([[0.0]]), np.array([[3.0]]), np.array([[2.0]]))
    assert dg[0, 0] == pytest.approx(2.0 * 3.0 * 0.5, rel=1e-15) and du[0, 0] == 0.0
    assert orc.swiglu_fwd(np.array([[40.0]]), np.array([[1.0]]))[0, 0] == pytest.approx(40.0, rel=1e-15)
    assert abs(orc.swiglu_fwd(np.array([[-40.0]]), np.array([[1.0]]))[0, 0]) < 1e-15
    # textbook value: SiLU(1) = 1 / (1 + e^-1)
    assert orc.swiglu_fwd(np.array([[1.0]]), np.array([[1.0]]))[0, 0] == pytest.approx(0.7310585786300049, rel=1e-15)
    rng = np.random.default_rng(3)
    g, u, dh = rng.normal(size=(3, 4)), rng.normal(size=(3, 4)), rng.normal(size=(3, 4))
    dg, du = orc.swiglu_bwd(g, u, dh)
    assert np.allclose(dg, _fd(lambda z: np.sum(dh * orc.swiglu_fwd(z, u)), g), rtol=1e-7, atol=1e-9)
    assert np.allclose(du, _fd(lambda z: np.sum(dh * orc.swiglu_fwd(g, z)), u), rtol=1e-7, atol=1e-9)


def test_rmsnorm_values_and_gradients():
    # a row of equal entries c normalises to sign(c) * w (eps = 0); scaling a row leaves y unchanged
    w = np.array([1.0, 2.0, -3.0, 0.5])
    assert np.allclose(orc.rmsnorm_fwd(np.full((1, 4), -2.5), w, 0.0), -w, rtol=1e-15)
    rng = np.random.default_rng(4)
    x, dy = rng.normal(size=(3, 4)), rng.normal(size=(3, 4))
    assert np.allclose(orc.rmsnorm_fwd(7.0 * x, w, 0.0), orc.rmsnorm_fwd(x, w, 0.0), rtol=1e-13)
    # hand value: x = (3, 4), w = 1: rms = sqrt(12.5)
    assert np.allclose(orc.rmsnorm_fwd(np.array([[3.0, 4.0]]), np.ones(2), 0.0), np.array([[3.0, 4.0]]) / np.sqrt(12.5))
    # eps enters under the root
    assert orc.rmsnorm_fwd(np.array([[0.0, 0.0]]), np.ones(2), 1e-6)[0, 0] == 0.0
    assert orc.rmsnorm_fwd(np.array([[1.0, 1.0]]), np.ones(2), 3.0)[0, 0] == pytest.approx(0.5, rel=1e-15)
    for eps in (0.0, 1e-5, 0.3):
        dx = orc.rmsnorm_bwd(x, w, dy, eps)
        assert np.allclose(dx, _fd(lambda z: np.sum(dy * orc.rmsnorm_fwd(z, w, eps)), x), rtol=1e-6, atol=1e-8)
    # scale invariance of y (eps = 0) makes dx orthogonal to x, row by row
    assert np.allclose(np.sum(orc.rmsnorm_bwd(x, w, dy, 0.0) * x, axis=1), 0.0, atol=1e-13)
