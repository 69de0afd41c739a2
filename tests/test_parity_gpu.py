"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same
seeded inputs, element by element.  Shapes span several tiles (128-row, 64/256-column tiles,
64-wide k-blocks) and ragged tails; the full-size workloads are in test_parity_full_gpu.py."""
import numpy as np
import pytest
import torch

from oracle import templora_oracle as orc
from paper_2401_11504_b200 import inputs
from parity_utils import (TOL, Guarded, assert_close, check_adam_steps, check_fwd_bwd, f64, hp32, make_state, oracle_fwd_bwd,
                          run_fwd_bwd, ill_conditioned_mask)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2401_11504_b200 import build
    build.build_library()
    from paper_2401_11504_b200 import binding
    assert torch.cuda.get_device_capability(0)[0] == 10, "these kernels are built for sm_100a only"
    binding.templora_set_kernel_path(0)
    return binding


@pytest.fixture
def generic_path(b):
    b.templora_set_kernel_path(1)
    yield b
    b.templora_set_kernel_path(0)


# ------------------------------------------------------------------ fp32 path (configuration 0)
def test_config0_fp32_fwd_bwd(b):
    c = inputs.CONFIGS[0]
    _, d_in, d_out = c["projections"][0]
    check_fwd_bwd(b, 0, "cfg0", c["T"], d_in, d_out, c["r"], c["s"], "f32")


@pytest.mark.parametrize("T,d_in,d_out,r", [(1, 8, 8, 1), (37, 100, 67, 5), (130, 70, 129, 8), (64, 64, 64, 16)])
def test_fp32_ragged_shapes(b, T, d_in, d_out, r):
    check_fwd_bwd(b, 1, f"f32-{T}-{d_in}-{d_out}-{r}", T, d_in, d_out, r, 2.0, "f32")


def test_fp32_options(b):
    # no dX, U recomputed in the backward, gradients accumulated onto existing contents
    check_fwd_bwd(b, 2, "f32-opts", 50, 96, 80, 8, 1.0, "f32", with_dX=False, save_U=False, accumulate=True)


# ------------------------------------------------------------------ bf16, tensor-core path
TC_SHAPES = [
    (128, 512, 512, 64),     # exactly one row tile
    (300, 328, 520, 24),     # ragged rows, d not a multiple of 64, rank below one k-block
    (1, 64, 72, 8),          # a single token
    (257, 1024, 264, 128),   # two rank k-blocks, ragged columns
    (640, 4096, 1024, 64),   # split-K in the skinny products
    (200, 136, 2048, 256),   # maximum rank
]


@pytest.mark.parametrize("T,d_in,d_out,r", TC_SHAPES)
def test_bf16_tensor_core_shapes(b, T, d_in, d_out, r):
    check_fwd_bwd(b, 3, f"tc-{T}-{d_in}-{d_out}-{r}", T, d_in, d_out, r, 2.0, "bf16")


def test_bf16_tensor_core_options(b):
    check_fwd_bwd(b, 4, "tc-opts", 384, 512, 768, 64, 1.0, "bf16", with_dX=False, save_U=False, accumulate=True)


def test_bf16_results_are_run_to_run_identical(b):
    host = inputs.make_linear(5, "det", 300, 512, 640, 64, dtype="bf16")
    a = run_fwd_bwd(b, host, 2.0, 300)
    c = run_fwd_bwd(b, host, 2.0, 300)
    for k in a:
        assert np.array_equal(a[k], c[k]), f"{k} differs between two runs"


def test_zero_B_gives_base_linear_and_zero_dA(b):
    got, ref, _ = check_fwd_bwd(b, 6, "zeroB", 200, 256, 320, 64, 2.0, "bf16", zero_B=True)
    assert not got["dA"].any()


# ------------------------------------------------------------------ bf16, generic path
@pytest.mark.parametrize("T,d_in,d_out,r", [(65, 100, 36, 5), (128, 512, 512, 64), (33, 200, 136, 8)])
def test_bf16_generic_path(generic_path, T, d_in, d_out, r):
    check_fwd_bwd(generic_path, 7, f"gen-{T}-{d_in}-{d_out}-{r}", T, d_in, d_out, r, 2.0, "bf16")


def test_bf16_unaligned_shape_takes_generic_path_automatically(b):
    check_fwd_bwd(b, 8, "auto-generic", 40, 100, 60, 4, 2.0, "bf16")


# ------------------------------------------------------------------ decode
@pytest.mark.parametrize("n", [1, 4, 16, 7])
@pytest.mark.parametrize("d_in,d_out,r", [(512, 640, 64), (4096, 1024, 64), (1000, 264, 16), (512, 384, 128), (256, 136, 256)])
def test_decode_matches_oracle(b, n, d_in, d_out, r):
    host = inputs.make_linear(9, f"dec-{n}-{d_in}-{d_out}", n, d_in, d_out, r, dtype="bf16")
    dev = {k: v.cuda() for k, v in host.items()}
    lin = b.linear_desc(dev["W0"], dev["A"], dev["B"], 2.0)
    guard = Guarded()
    ws = guard.workspace(b.templora_workspace_bytes(lin, 16))
    y = guard.empty((n, d_out), torch.bfloat16)
    b.templora_decode_fwd(lin, dev["x"], y, ws)
    assert b.templora_read_device_status(ws)[0] == 0
    guard.check("after templora_decode_fwd")
    ref = orc.decode_fwd(f64(host["x"]), f64(host["W0"]), f64(host["A"]), f64(host["B"]), 2.0)
    assert_close("decode y", f64(y), ref, TOL["bf16"])


def test_decode_fp32_and_generic(generic_path):
    b = generic_path
    for dtype in ("f32", "bf16"):
        host = inputs.make_linear(10, "dec-gen-" + dtype, 4, 96, 72, 8, dtype=dtype)
        dev = {k: v.cuda() for k, v in host.items()}
        lin = b.linear_desc(dev["W0"], dev["A"], dev["B"], 2.0)
        ws = b.alloc_workspace(b.templora_workspace_bytes(lin, 16))
        y = torch.empty((4, 72), dtype=host["x"].dtype, device="cuda")
        b.templora_decode_fwd(lin, dev["x"], y, ws)
        ref = orc.decode_fwd(f64(host["x"]), f64(host["W0"]), f64(host["A"]), f64(host["B"]), 2.0)
        assert_close("decode y", f64(y), ref, TOL[dtype])


def test_decode_block_matches_oracle(b):
    # eleven independent projections in one call: more than one group of eight, mixed shapes,
    # one of them (d_in = 100) outside the tensor-core path
    shapes = [(512, 640, 64), (512, 640, 64), (1024, 264, 16), (2048, 512, 64), (100, 60, 4)] * 2 + [(4096, 1024, 64)]
    for n in (1, 5, 16):
        hosts = [inputs.make_linear(14, f"decblk-{n}-{i}", n, di, do, r, dtype="bf16") for i, (di, do, r) in enumerate(shapes)]
        devs = [{k: v.cuda() for k, v in h.items()} for h in hosts]
        lins = [b.linear_desc(d["W0"], d["A"], d["B"], 2.0) for d in devs]
        guard = Guarded()
        ys = [guard.empty((n, do), torch.bfloat16) for _, do, _ in shapes]
        ws = guard.workspace(b.templora_decode_block_workspace_bytes(lins))
        args = b.DecodeBlockArgs(lins, [d["x"] for d in devs], ys)
        b.templora_decode_block_fwd(args, ws)
        assert b.templora_read_device_status(ws)[0] == 0
        guard.check(f"after templora_decode_block_fwd n={n}")
        for i, h in enumerate(hosts):
            ref = orc.decode_fwd(f64(h["x"]), f64(h["W0"]), f64(h["A"]), f64(h["B"]), 2.0)
            assert_close(f"decode block y{i} n={n}", f64(ys[i]), ref, TOL["bf16"])


def test_single_cta_tensor_core_path(b):
    # kernel path 2: frozen-weight GEMMs on single-CTA 128 x 256 tiles instead of CTA pairs
    b.templora_set_kernel_path(2)
    try:
        check_fwd_bwd(b, 15, "tc-single", 300, 328, 520, 24, 2.0, "bf16")
        check_fwd_bwd(b, 15, "tc-single2", 640, 1024, 768, 64, 2.0, "bf16")
    finally:
        b.templora_set_kernel_path(0)


# ------------------------------------------------------------------ AdamW
def _adamw_case(b, n, dtype, steps, hp, seed):
    hp = hp32(hp)
    g = torch.Generator().manual_seed(seed)
    p0 = (torch.randn(n, generator=g) * 0.02).float()
    grads = [torch.randn(n, generator=g).float() * (0.5 + k) for k in range(steps)]
    p, m, v = p0.cuda(), torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    work = torch.zeros(n, dtype=torch.bfloat16, device="cuda") if dtype == "bf16" else None
    rp, rm, rv = f64(p0), np.zeros(n), np.zeros(n)
    for t in range(1, steps + 1):
        gd = grads[t - 1].cuda()
        before = f64(p)
        b.templora_adamw_step([b.param_desc(p, m, v, gd, work)], step=t,
                              work_dtype=b.BF16 if dtype == "bf16" else b.F32, **hp)
        torch.cuda.synchronize()
        rp_new, rm, rv = orc.adamw_step(rp, f64(grads[t - 1]), rm, rv, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
                                        hp["weight_decay"], t)
        assert_close("p", f64(p), rp_new, 1e-5)
        assert_close("m", f64(m), rm, 1e-5)
        assert_close("v", f64(v), rv, 1e-5)
        # the step itself: |dp| ~ lr is far below |p|, so compare the deltas; fp32 storage of p
        # adds half an ulp of |p| to each side
        d_gpu, d_ref = f64(p) - before, rp_new - rp
        bound = 1e-5 * np.abs(d_ref).max() + 2.0 ** -23 * np.abs(rp).max()
        assert np.abs(d_gpu - d_ref).max() <= bound
        assert np.abs(d_ref).max() > 0
        if work is not None:
            assert np.array_equal(f64(work), orc.round_bf16(f64(p).astype(np.float32)))
        # the oracle continues from the fp32 state the device holds (storage rounding is not error)
        rp, rm, rv = f64(p), f64(m), f64(v)


@pytest.mark.parametrize("n", [1, 7, 4096, 64 * 4096 + 3])
def test_adamw_matches_oracle(b, n):
    _adamw_case(b, n, "bf16", 3, dict(inputs.ADAMW), 11)
    _adamw_case(b, n, "f32", 2, dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1), 12)


def test_adamw_many_tensors_one_call(b):
    hp = hp32(inputs.ADAMW)
    sizes = [5, 64 * 512, 3, 512 * 64, 1000] * 30      # 150 tensors: several launches of 64
    g = torch.Generator().manual_seed(13)
    ps = [(torch.randn(n, generator=g) * 0.02).float().cuda() for n in sizes]
    gs = [torch.randn(n, generator=g).float().cuda() for n in sizes]
    ms = [torch.zeros(n, device="cuda") for n in sizes]
    vs = [torch.zeros(n, device="cuda") for n in sizes]
    ws_ = [torch.zeros(n, dtype=torch.bfloat16, device="cuda") for n in sizes]
    p0 = [f64(p) for p in ps]
    b.templora_adamw_step([b.param_desc(p, m, v, gd, w) for p, m, v, gd, w in zip(ps, ms, vs, gs, ws_)], step=1, **hp)
    torch.cuda.synchronize()
    for i in (0, 1, 63, 64, 65, 149):
        rp, rm, rv = orc.adamw_step(p0[i], f64(gs[i]), 0 * p0[i], 0 * p0[i], hp["lr"], hp["beta1"], hp["beta2"],
                                    hp["eps"], hp["weight_decay"], 1)
        assert_close("p", f64(ps[i]), rp, 1e-5)
        assert_close("v", f64(vs[i]), rv, 1e-5)
        assert np.array_equal(f64(ws_[i]), orc.round_bf16(f64(ps[i]).astype(np.float32)))


# ------------------------------------------------------------------ update_block
def _make_update_args(b, hosts, dtype, s, with_dX):
    """Fresh device tensors, optimizer state and marshalled arguments for one templora_update_block* call."""
    devs = [{k: v.cuda() for k, v in h.items()} for h in hosts]
    states = [make_state(h, dtype) for h in hosts]
    lins, As, Bs, ys, dXs = [], [], [], [], []
    for d, st in zip(devs, states):
        a = st["A"]["work"] if dtype == "bf16" else st["A"]["master"]
        bb = st["B"]["work"] if dtype == "bf16" else st["B"]["master"]
        lins.append(b.linear_desc(d["W0"], a, bb, s))
        As.append(b.param_desc(st["A"]["master"], st["A"]["m"], st["A"]["v"], st["A"]["grad"], st["A"]["work"]))
        Bs.append(b.param_desc(st["B"]["master"], st["B"]["m"], st["B"]["v"], st["B"]["grad"], st["B"]["work"]))
        ys.append(torch.full_like(d["dY"], float("nan")))
        dXs.append(torch.full_like(d["x"], float("nan")) if with_dX else None)
    return dict(devs=devs, states=states, lins=lins, As=As, Bs=Bs, ys=ys, dXs=dXs)


def _step_by_step(b, u, hosts, dtype, s, T, batch, epochs, hp, warmup, with_dX, ws):
    """The same update taken one optimizer step per call (the row slice of that step, epochs = 1, the step count
    carried over), on fresh state u.  After every call: the device's gradients against the oracle's backward
    from the device's own current working copies, and the oracle's AdamW fed with the device's gradients, moments
    and parameters against the device's new parameters: tightly, because both sides then get the same gradient."""
    tol = TOL[dtype]
    rows_per = T if batch is None else batch
    k = 0
    for _ in range(epochs):
        for r0 in range(0, T, rows_per):
            r1 = min(r0 + rows_per, T)
            sl = lambda ts: [None if t is None else t[r0:r1] for t in ts]
            args = b.UpdateBlockArgs(u["lins"], u["As"], u["Bs"], sl([d["x"] for d in u["devs"]]),
                                     sl([d["dY"] for d in u["devs"]]), sl(u["ys"]), sl(u["dXs"]) if with_dX else None)
            before = [{nm: {q: f64(st[nm][q]) for q in ("master", "m", "v")} for nm in ("A", "B")} for st in u["states"]]
            work = [{nm: f64(st[nm]["work"] if dtype == "bf16" else st[nm]["master"]) for nm in ("A", "B")}
                    for st in u["states"]]
            k1 = b.templora_update_block_warmup(args, r1 - r0, 1, hp["lr"], warmup, hp["beta1"], hp["beta2"], hp["eps"],
                                                hp["weight_decay"], k, ws)
            assert k1 == k + 1 and b.templora_read_device_status(ws)[0] == 0
            k = k1
            lr_k = float(np.float32(orc.lr_at_step(hp["lr"], k, warmup)))
            for i, (h, st) in enumerate(zip(hosts, u["states"])):
                _, dA, dB = orc.linear_bwd(f64(h["x"])[r0:r1], f64(h["dY"])[r0:r1], f64(h["W0"]), work[i]["A"], work[i]["B"], s)
                for nm, g_ref in (("A", dA), ("B", dB)):
                    g_dev = f64(st[nm]["grad"])
                    assert_close(f"step {k} d{nm}{i}", g_dev, g_ref, tol)
                    p0 = before[i][nm]["master"]
                    p1, m1, v1 = orc.adamw_step(p0, g_dev, before[i][nm]["m"], before[i][nm]["v"], lr_k, hp["beta1"],
                                                hp["beta2"], hp["eps"], hp["weight_decay"], k)
                    got = f64(st[nm]["master"])
                    tight = 1e-5 * np.abs(p1 - p0).max() + 2.0 ** -23 * np.abs(p1).max()
                    assert np.abs((got - p0) - (p1 - p0)).max() <= tight, f"step {k} {nm}{i}: optimizer arithmetic"
                    assert_close(f"step {k} m{nm}{i}", f64(st[nm]["m"]), m1, 1e-5)
                    assert_close(f"step {k} v{nm}{i}", f64(st[nm]["v"]), v1, 1e-5)
    return k


def _update_block_case(b, dtype, shapes, T, r, s, epochs, hp, seed, with_dX=True, batch=None, warmup=0):
    hp = hp32(hp)
    hosts = [inputs.make_linear(seed, f"ub{i}", T, di, do, r, dtype=dtype) for i, (di, do) in enumerate(shapes)]
    u = _make_update_args(b, hosts, dtype, s, with_dX)
    devs, states, lins, ys, dXs = u["devs"], u["states"], u["lins"], u["ys"], u["dXs"]
    ws = b.alloc_workspace(b.templora_update_block_workspace_bytes(lins, T))
    args = b.UpdateBlockArgs(lins, u["As"], u["Bs"], [d["x"] for d in devs], [d["dY"] for d in devs], ys,
                             dXs if with_dX else None)
    if warmup:
        step = b.templora_update_block_warmup(args, batch or T, epochs, hp["lr"], warmup, hp["beta1"], hp["beta2"],
                                              hp["eps"], hp["weight_decay"], 0, ws)
    elif batch is None:
        step = b.templora_update_block(args, epochs, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
                                       hp["weight_decay"], 0, ws)
    else:
        step = b.templora_update_block_batched(args, batch, epochs, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
                                               hp["weight_decay"], 0, ws)
    assert b.templora_read_device_status(ws)[0] == 0
    n_steps = epochs * (1 if batch is None else -(-T // batch))
    assert step == n_steps

    # The same update one optimizer step per call, checked tightly at every step, must end in the very same
    # bits: so every step of the multi-step call above is covered by a well-conditioned comparison, whatever
    # the conditioning of the end-to-end comparison with the oracle below.
    u2 = _make_update_args(b, hosts, dtype, s, with_dX)
    assert _step_by_step(b, u2, hosts, dtype, s, T, batch, epochs, hp, warmup, with_dX, ws) == n_steps
    for i, (st, st2) in enumerate(zip(states, u2["states"])):
        for nm in ("A", "B"):
            for q in ("master", "m", "v", "grad") + (("work",) if dtype == "bf16" else ()):
                assert torch.equal(st[nm][q], st2[nm][q]), f"{nm}{i}.{q}: one call and step-by-step calls differ"
        assert torch.equal(ys[i], u2["ys"][i])
        if with_dX:
            assert torch.equal(dXs[i], u2["dXs"][i])

    projs = [dict(x=f64(h["x"]), dY=f64(h["dY"]), W0=f64(h["W0"]), s=s, A_master=f64(h["A"]), B_master=f64(h["B"]))
             for h in hosts]
    grad_log = []
    ref, rstep = orc.update_block(projs, epochs, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"],
                                  bf16_work=(dtype == "bf16"), batch=batch, warmup_steps=warmup,
                                  lr_round=lambda v: float(np.float32(v)), grad_log=grad_log)
    assert rstep == step
    lrs = [float(np.float32(orc.lr_at_step(hp["lr"], k + 1, warmup))) for k in range(n_steps)]
    fracs = {}
    tol = TOL[dtype]
    for i, (q, st) in enumerate(zip(ref, states)):
        assert_close(f"y{i}", f64(ys[i]), q["y"], tol)
        if with_dX:
            assert_close(f"dX{i}", f64(dXs[i]), q["dX"], tol)
        assert_close(f"dA{i}", f64(st["A"]["grad"]), q["dA"], tol)
        assert_close(f"dB{i}", f64(st["B"]["grad"]), q["dB"], tol)
        for nm in ("A", "B"):
            # End to end against the oracle: the movement of the parameters (|delta| ~ steps * lr << |p|).
            # Adam's step is sign-like (lr * g / (|g| + eps) at step 1) and so ill-conditioned where a gradient
            # is within its own tolerance of zero or changes between steps; ill_conditioned_mask finds those
            # elements from the oracle's per-step gradients, and only there may the two sides differ.
            p0 = f64(hosts[i][nm])
            got = f64(st[nm]["master"])
            mask = ill_conditioned_mask(grad_log, i, nm, p0, hp, tol, lrs=lrs)
            fracs[f"{nm}{i}"] = (check_adam_steps(f"{nm}{i}", p0, got, q[nm + "_master"], mask, tol, n_steps, hp["lr"],
                                                  max_frac=0.02 if dtype == "bf16" else 1e-3), float(mask.mean()))
            assert_close(f"m{nm}{i}", f64(st[nm]["m"]), q["m" + nm], tol)
            assert_close(f"v{nm}{i}", f64(st[nm]["v"]), q["v" + nm], 2 * tol)   # v is quadratic in g
            if dtype == "bf16":
                assert np.array_equal(f64(st[nm]["work"]), orc.round_bf16(f64(st[nm]["master"]).astype(np.float32)))
    print("optimizer steps outside the tight bound / ill-conditioned under the gradient tolerance (fractions):",
          {k: f"{v[0]:.4f} / {v[1]:.4f}" for k, v in fracs.items()})


def test_update_block_fp32_config0(b):
    c = inputs.CONFIGS[0]
    _update_block_case(b, "f32", [(512, 512)], c["T"], c["r"], c["s"], 1, dict(inputs.ADAMW), 0)


def test_update_block_bf16_two_epochs(b):
    shapes = [(256, 256), (256, 256), (256, 704), (704, 256)]
    _update_block_case(b, "bf16", shapes, 200, 64, 2.0, 2, dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8,
                                                                 weight_decay=0.0), 21)


def test_update_block_more_projections_than_one_group(b):
    shapes = [(128, 192)] * 5 + [(192, 128)] * 6
    _update_block_case(b, "bf16", shapes, 130, 16, 2.0, 1, dict(inputs.ADAMW), 22, with_dX=False)


def test_update_block_generic_path(generic_path):
    _update_block_case(generic_path, "bf16", [(100, 60), (60, 100)], 33, 4, 2.0, 2,
                       dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01), 23)


@pytest.mark.parametrize("T,batch", [(512, 256), (600, 256), (384, 128)])
def test_update_block_batched_bf16(b, T, batch):
    # chunk cut into batches: epochs * ceil(T / batch) optimizer steps, ragged last batch included
    shapes = [(256, 384), (384, 256), (256, 256)]
    _update_block_case(b, "bf16", shapes, T, 64, 2.0, 2, dict(lr=2e-4, beta1=0.9, beta2=0.999, eps=1e-8,
                                                               weight_decay=0.0), 26, batch=batch)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_update_block_with_lr_warmup(b, dtype):
    # six optimizer steps (2 epochs x 3 batches), the rate rising linearly over the first four
    shapes = [(256, 384), (384, 256)] if dtype == "bf16" else [(96, 80), (80, 64)]
    r = 64 if dtype == "bf16" else 8
    _update_block_case(b, dtype, shapes, 384 if dtype == "bf16" else 90, r, 2.0, 2,
                       dict(lr=2e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01), 28,
                       batch=128 if dtype == "bf16" else 30, warmup=4)


def test_update_block_batched_fp32(b):
    _update_block_case(b, "f32", [(96, 80)], 70, 8, 2.0, 1, dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8,
                                                                 weight_decay=0.01), 27, batch=32)


def test_update_block_zero_epochs_is_a_no_op(b):
    host = inputs.make_linear(24, "noop", 16, 64, 64, 8, dtype="bf16")
    d = {k: v.cuda() for k, v in host.items()}
    st = make_state(host, "bf16")
    lin = b.linear_desc(d["W0"], st["A"]["work"], st["B"]["work"], 2.0)
    A = b.param_desc(st["A"]["master"], st["A"]["m"], st["A"]["v"], st["A"]["grad"], st["A"]["work"])
    Bp = b.param_desc(st["B"]["master"], st["B"]["m"], st["B"]["v"], st["B"]["grad"], st["B"]["work"])
    y = torch.zeros_like(d["dY"])
    ws = b.alloc_workspace(b.templora_update_block_workspace_bytes([lin], 16))
    args = b.UpdateBlockArgs([lin], [A], [Bp], [d["x"]], [d["dY"]], [y])
    assert b.templora_update_block(args, 0, 1e-3, 0.9, 0.999, 1e-8, 0.0, 5, ws) == 5
    torch.cuda.synchronize()
    assert np.array_equal(f64(st["A"]["master"]), f64(host["A"]))


# ------------------------------------------------------------------ errors that need a device
def test_short_workspace_is_rejected(b):
    host = inputs.make_linear(25, "short", 256, 512, 512, 64, dtype="bf16")
    d = {k: v.cuda() for k, v in host.items()}
    lin = b.linear_desc(d["W0"], d["A"], d["B"], 2.0)
    ws = b.alloc_workspace(2048)
    y = torch.empty((256, 512), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(b.TemploraError) as e:
        b.templora_linear_fwd(lin, d["x"], y, ws)
    assert e.value.code == b.ERR_WORKSPACE


# ------------------------------------------------------------------ failure detection
def test_a_wait_that_nothing_satisfies_times_out_and_the_context_survives(b):
    import time
    ws = b.alloc_workspace(4096)
    t0 = time.perf_counter()
    b.templora_selftest_bounded_wait(ws, limit_ms=50)
    code, where = b.templora_read_device_status(ws)
    dt = time.perf_counter() - t0
    assert code == b.ERR_TIMEOUT and where == 900
    assert 0.04 < dt < 2.0
    # the stream and the context are still good: a normal call right after gives a correct result
    ws.zero_()
    check_fwd_bwd(b, 50, "after-timeout", 130, 256, 264, 16, 2.0, "bf16")
    # argument checks
    with pytest.raises(b.TemploraError):
        b.templora_selftest_bounded_wait(ws, limit_ms=5000)


# ------------------------------------------------------------------ decode: both forms, repeated calls
def _decode_case(b, seed, tag, n, d_in, d_out, r, ws=None):
    host = inputs.make_linear(seed, tag, n, d_in, d_out, r, dtype="bf16")
    dev = {k: v.cuda() for k, v in host.items()}
    lin = b.linear_desc(dev["W0"], dev["A"], dev["B"], 2.0)
    guard = Guarded()
    if ws is None:
        ws = guard.workspace(b.templora_workspace_bytes(lin, 16))
    y = guard.empty((n, d_out), torch.bfloat16)
    b.templora_decode_fwd(lin, dev["x"], y, ws)
    assert b.templora_read_device_status(ws)[0] == 0
    guard.check(f"after templora_decode_fwd ({tag})")
    ref = orc.decode_fwd(f64(host["x"]), f64(host["W0"]), f64(host["A"]), f64(host["B"]), 2.0)
    assert_close(f"decode y {tag}", f64(y), ref, TOL["bf16"])
    return ws


@pytest.mark.parametrize("n", [1, 5, 16])
def test_decode_two_kernel_form(b, n):
    # kernel path 2 keeps the split-K slabs + finish kernel form of the decode-time forward
    b.templora_set_kernel_path(2)
    try:
        _decode_case(b, 21, f"dec2k-{n}", n, 2048, 1152, 64)
        _decode_case(b, 21, f"dec2k-r16-{n}", n, 1000, 264, 16)
    finally:
        b.templora_set_kernel_path(0)


def test_decode_repeated_calls_share_a_workspace(b):
    # s*u of an earlier call stays in the workspace; every call must wait for its own (the ready flags are
    # cleared at the end of each launch) and the item counter must be re-armed between calls, also across the two forms
    d_in, d_out, r = 4096, 1280, 64
    host = inputs.make_linear(22, "dec-rep", 16, d_in, d_out, r, dtype="bf16")
    lin_probe = b.linear_desc(host["W0"].cuda(), host["A"].cuda(), host["B"].cuda(), 2.0)
    ws = b.alloc_workspace(b.templora_workspace_bytes(lin_probe, 16))
    for rep in range(6):
        if rep == 3:
            b.templora_set_kernel_path(2)
        try:
            _decode_case(b, 23 + rep, f"dec-rep-{rep}", (1, 16, 4, 7, 2, 16)[rep], d_in, d_out, r, ws=ws)
        finally:
            b.templora_set_kernel_path(0)


def test_decode_block_replayed_from_a_cuda_graph(b):
    # the launch depends on nothing the host hands in per call (ready flags and the item counter are re-armed on the
    # device), so a decode step recorded once can be replayed: new inputs in the same buffers, same results as a
    # direct call and as the oracle
    shapes = [(1024, 768, 64), (1024, 768, 64), (768, 1024, 32)]
    n = 4
    hosts = [inputs.make_linear(61, f"graph{i}", n, di, do, r, dtype="bf16") for i, (di, do, r) in enumerate(shapes)]
    devs = [{k: v.cuda() for k, v in h.items()} for h in hosts]
    lins = [b.linear_desc(d["W0"], d["A"], d["B"], 2.0) for d in devs]
    xs = [d["x"].clone() for d in devs]
    ys = [torch.empty((n, do), dtype=torch.bfloat16, device="cuda") for _, do, _ in shapes]
    ws = b.alloc_workspace(b.templora_decode_block_workspace_bytes(lins))
    args = b.DecodeBlockArgs(lins, xs, ys)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        b.templora_decode_block_fwd(args, ws, stream=side)      # first call outside the capture: one-time set-up
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        b.templora_decode_block_fwd(args, ws, stream=torch.cuda.current_stream())
    for rep in range(3):
        new_x = [inputs.make_tensor(62 + rep, f"graph{i}", "x", (n, di), "normal", 1.0, "bf16", "cpu") for i, (di, _, _) in enumerate(shapes)]
        for x, nx in zip(xs, new_x):
            x.copy_(nx.cuda())
        for y in ys:
            y.fill_(float("nan"))
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert b.templora_read_device_status(ws)[0] == 0
        for i, h in enumerate(hosts):
            ref = orc.decode_fwd(f64(new_x[i]), f64(h["W0"]), f64(h["A"]), f64(h["B"]), 2.0)
            assert_close(f"graph replay {rep} y{i}", f64(ys[i]), ref, TOL["bf16"])


# ------------------------------------------------------------------ projections that share their input
def _shared_input_case(b, dtype, d_in, d_outs, T, r, seed, dropout_p=0.0, epochs=1):
    """q, k, v style: one x, one dX buffer for all projections; dX must be the sum of the input gradients."""
    hp = hp32(dict(lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0))
    hosts = [inputs.make_linear(seed, f"sh{i}", T, d_in, do, r, dtype=dtype) for i, do in enumerate(d_outs)]
    x_host = hosts[0]["x"]
    x_dev = x_host.cuda()
    devs = [{k: v.cuda() for k, v in h.items()} for h in hosts]
    states = [make_state(h, dtype) for h in hosts]
    dX = torch.full_like(x_dev, float("nan"))
    lins, As, Bs, ys = [], [], [], []
    for i, (d, st) in enumerate(zip(devs, states)):
        a = st["A"]["work"] if dtype == "bf16" else st["A"]["master"]
        bb = st["B"]["work"] if dtype == "bf16" else st["B"]["master"]
        lins.append(b.linear_desc(d["W0"], a, bb, 2.0, dropout_p=dropout_p, dropout_seed=1000 + i, input_group=7))
        As.append(b.param_desc(st["A"]["master"], st["A"]["m"], st["A"]["v"], st["A"]["grad"], st["A"]["work"]))
        Bs.append(b.param_desc(st["B"]["master"], st["B"]["m"], st["B"]["v"], st["B"]["grad"], st["B"]["work"]))
        ys.append(torch.full_like(d["dY"], float("nan")))
    ws = b.alloc_workspace(b.templora_update_block_workspace_bytes(lins, T))
    n = len(hosts)
    args = b.UpdateBlockArgs(lins, As, Bs, [x_dev] * n, [d["dY"] for d in devs], ys, [dX] * n)
    step = b.templora_update_block(args, epochs, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"], 0, ws)
    assert b.templora_read_device_status(ws)[0] == 0 and step == epochs
    projs = [dict(x=f64(x_host), dY=f64(h["dY"]), W0=f64(h["W0"]), s=2.0, A_master=f64(h["A"]), B_master=f64(h["B"]),
                  dX_to=None if i == 0 else 0, dropout_seed=1000 + i) for i, h in enumerate(hosts)]
    ref, _ = orc.update_block(projs, epochs, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"],
                              bf16_work=(dtype == "bf16"), dropout_p=dropout_p)
    tol = TOL[dtype]
    assert_close("summed dX", f64(dX), ref[0]["dX"], tol)
    for i, (q, st) in enumerate(zip(ref, states)):
        assert_close(f"y{i}", f64(ys[i]), q["y"], tol)
        assert_close(f"dA{i}", f64(st["A"]["grad"]), q["dA"], tol)
        assert_close(f"dB{i}", f64(st["B"]["grad"]), q["dB"], tol)


@pytest.mark.parametrize("d_outs", [(384, 256, 256), (640, 640)])
def test_shared_input_summed_dx_bf16(b, d_outs):
    _shared_input_case(b, "bf16", 512, d_outs, 300, 64, 31)


def test_shared_input_summed_dx_two_epochs_and_single_cta_tiles(b):
    _shared_input_case(b, "bf16", 256, (256, 384, 128), 200, 16, 32, epochs=2)
    b.templora_set_kernel_path(2)
    try:
        _shared_input_case(b, "bf16", 512, (384, 256, 256), 300, 64, 31)
    finally:
        b.templora_set_kernel_path(0)


def test_shared_input_summed_dx_with_dropout(b):
    _shared_input_case(b, "bf16", 512, (384, 256, 256), 300, 64, 33, dropout_p=0.1)


def test_shared_input_summed_dx_fp32_and_generic(b, generic_path):
    _shared_input_case(generic_path, "f32", 96, (80, 64, 72), 50, 8, 34)
    _shared_input_case(generic_path, "bf16", 128, (96, 64), 70, 8, 35)


def test_shared_dx_needs_equal_input_width(b):
    hosts = [inputs.make_linear(36, f"bad{i}", 32, di, 64, 8, dtype="bf16") for i, di in enumerate((64, 128))]
    devs = [{k: v.cuda() for k, v in h.items()} for h in hosts]
    states = [make_state(h, "bf16") for h in hosts]
    lins = [b.linear_desc(d["W0"], st["A"]["work"], st["B"]["work"], 2.0, input_group=1) for d, st in zip(devs, states)]
    As = [b.param_desc(st["A"]["master"], st["A"]["m"], st["A"]["v"], st["A"]["grad"], st["A"]["work"]) for st in states]
    Bs = [b.param_desc(st["B"]["master"], st["B"]["m"], st["B"]["v"], st["B"]["grad"], st["B"]["work"]) for st in states]
    ys = [torch.empty_like(d["dY"]) for d in devs]
    dX = torch.empty((32, 128), dtype=torch.bfloat16, device="cuda")
    ws = b.alloc_workspace(b.templora_update_block_workspace_bytes(lins, 32))
    args = b.UpdateBlockArgs(lins, As, Bs, [d["x"] for d in devs], [d["dY"] for d in devs], ys, [dX, dX])
    with pytest.raises(b.TemploraError):
        b.templora_update_block(args, 1, 1e-4, 0.9, 0.999, 1e-8, 0.0, 0, ws)


def test_decode_block_under_a_tight_sm_cap(b):
    # eight SMs fit fewer clusters than the call has projections: the one-kernel form steps aside for the
    # two-kernel form, and a cap of 24 SMs runs the one-kernel form on few clusters; both must match
    shapes = [(512, 640, 64)] * 4 + [(1024, 384, 64)] * 3
    n = 4
    hosts = [inputs.make_linear(37, f"cap-{i}", n, di, do, r, dtype="bf16") for i, (di, do, r) in enumerate(shapes)]
    devs = [{k: v.cuda() for k, v in h.items()} for h in hosts]
    lins = [b.linear_desc(d["W0"], d["A"], d["B"], 2.0) for d in devs]
    ws = b.alloc_workspace(b.templora_decode_block_workspace_bytes(lins))
    stream = torch.cuda.Stream()
    for cap in (8, 24, 0):
        b.templora_set_stream_sm_limit(stream, cap)
        ys = [torch.full((n, do), float("nan"), dtype=torch.bfloat16, device="cuda") for _, do, _ in shapes]
        args = b.DecodeBlockArgs(lins, [d["x"] for d in devs], ys)
        torch.cuda.synchronize()
        b.templora_decode_block_fwd(args, ws, stream=stream)
        stream.synchronize()
        assert b.templora_read_device_status(ws, stream=stream)[0] == 0
        for i, h in enumerate(hosts):
            ref = orc.decode_fwd(f64(h["x"]), f64(h["W0"]), f64(h["A"]), f64(h["B"]), 2.0)
            assert_close(f"cap {cap} y{i}", f64(ys[i]), ref, TOL["bf16"])
    b.templora_set_stream_sm_limit(stream, 0)
