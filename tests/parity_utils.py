"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI on seeded
inputs, run the fp64 oracle on the same tensors, compare per output tensor.

Tolerances (per output tensor, normwise):  max|gpu - ref| <= tol * max|ref| with
tol = 1e-2 for bf16 storage with fp32 accumulation and 1e-5 for the fp32 path.
"""
import numpy as np
import torch

from oracle import templora_oracle as orc
from paper_2401_11504_b200 import inputs

TOL = {"f32": 1e-5, "bf16": 1e-2}


def hp32(hp):
    """Optimizer hyper-parameters as the C ABI receives them: rounded to fp32 (1 - beta2 changes by
    1.3e-5 relative when 0.999 is rounded to fp32; both sides must see the same value)."""
    return {k: float(np.float32(v)) for k, v in hp.items()}


def tdtype(dtype):
    return {"f32": torch.float32, "bf16": torch.bfloat16}[dtype]


def assert_close(name, got, ref, tol):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, f"{name}: shape {got.shape} vs {ref.shape}"
    assert np.isfinite(got).all(), f"{name}: non-finite values"
    scale = np.abs(ref).max()
    err = np.abs(got - ref).max()
    assert err <= tol * scale + 1e-30, f"{name}: max|err| {err:.3e} > {tol:g} * max|ref| {scale:.3e}"
    return err / max(scale, 1e-300)


def f64(t):
    return inputs.to_f64(t)


class Guarded:
    """Device buffers with canary words on both sides.  compute-sanitizer is not available where these tests run,
    so writes past the ends of an output or of the workspace are caught this way: every buffer handed to the
    library sits inside a larger allocation whose margins hold a fixed bit pattern, and check() requires the
    margins to be bit-for-bit intact afterwards.  (NaN-filled outputs show elements that were NOT written; the
    margins show writes that should not have happened.)"""
    MARGIN = 4096          # bytes on each side; a multiple of 1024 so that a workspace keeps its alignment
    PATTERN = 0xA5

    def __init__(self):
        self.items = []

    def empty(self, shape, dtype, fill=float("nan")):
        n = int(np.prod(shape))
        esize = torch.empty((), dtype=dtype).element_size()
        raw = torch.full((2 * self.MARGIN + n * esize,), self.PATTERN, dtype=torch.uint8, device="cuda")
        view = raw[self.MARGIN:self.MARGIN + n * esize].view(dtype).view(*shape)
        view.fill_(fill)
        self.items.append((raw, n * esize))
        return view

    def workspace(self, nbytes):
        nbytes = int(nbytes)
        raw = torch.full((2 * self.MARGIN + nbytes,), self.PATTERN, dtype=torch.uint8, device="cuda")
        view = raw[self.MARGIN:self.MARGIN + nbytes]
        view.zero_()
        assert view.data_ptr() % 256 == 0
        self.items.append((raw, nbytes))
        return view

    def check(self, what=""):
        for k, (raw, nbytes) in enumerate(self.items):
            lo, hi = raw[:self.MARGIN], raw[self.MARGIN + nbytes:]
            assert bool((lo == self.PATTERN).all()), f"{what}: buffer {k}: bytes BEFORE its start were overwritten"
            assert bool((hi == self.PATTERN).all()), f"{what}: buffer {k}: bytes PAST its end were overwritten"


def run_fwd_bwd(b, host, s, T, with_dX=True, save_U=True, accumulate=False, dropout=None):
    """host: dict of CPU tensors (x, W0, A, B, dY).  Returns GPU outputs as float64 numpy."""
    dev = {k: v.cuda() for k, v in host.items()}
    d_out, d_in = host["W0"].shape
    r = host["A"].shape[0]
    dkw = {} if dropout is None else dict(dropout_p=dropout[0], dropout_seed=dropout[1], dropout_offset=dropout[2])
    lin = b.linear_desc(dev["W0"], dev["A"], dev["B"], s, **dkw)
    guard = Guarded()       # every output and the workspace carry canary margins
    ws = guard.workspace(b.templora_workspace_bytes(lin, T))
    dt = host["x"].dtype
    y = guard.empty((T, d_out), dt)
    dX = guard.empty((T, d_in), dt) if with_dX else None
    U = guard.empty((T, r), torch.float32) if save_U else None
    init = 1.0 if accumulate else float("nan")
    dA = guard.empty((r, d_in), torch.float32, init)
    dB = guard.empty((d_out, r), torch.float32, init)
    b.templora_linear_fwd(lin, dev["x"], y, ws, U_save=U)
    guard.check("after templora_linear_fwd")
    b.templora_linear_bwd(lin, dev["x"], dev["dY"], dX, dA, dB, ws, U_saved=U, accumulate=accumulate)
    guard.check("after templora_linear_bwd")
    code, where = b.templora_read_device_status(ws)
    assert code == 0, f"device status {code} at {where}"
    out = dict(y=f64(y), dA=f64(dA), dB=f64(dB))
    if with_dX:
        out["dX"] = f64(dX)
    if save_U:
        out["U"] = f64(U)
    return out


def oracle_fwd_bwd(host, s, dropout=None):
    x, W0, A, B, dY = (f64(host[k]) for k in ("x", "W0", "A", "B", "dY"))
    keep, p = None, 0.0
    if dropout is not None:
        p = float(np.float32(dropout[0]))        # p crosses the ABI as fp32
        keep = orc.dropout_keep(dropout[1], dropout[2], x.shape[0], x.shape[1], p)
    y, U = orc.linear_fwd(x, W0, A, B, s, keep, p)
    dX, dA, dB = orc.linear_bwd(x, dY, W0, A, B, s, keep, p)
    return dict(y=y, U=U, dX=dX, dA=dA, dB=dB)


def check_fwd_bwd(b, seed, tag, T, d_in, d_out, r, s, dtype, **kw):
    host = inputs.make_linear(seed, tag, T, d_in, d_out, r, dtype=dtype, zero_B=kw.pop("zero_B", False))
    got = run_fwd_bwd(b, host, s, T, **kw)
    ref = oracle_fwd_bwd(host, s, kw.get("dropout"))
    if kw.get("accumulate"):
        ref["dA"] = ref["dA"] + 1.0
        ref["dB"] = ref["dB"] + 1.0
    errs = {}
    for k in got:
        errs[k] = assert_close(f"{tag}:{k}", got[k], ref[k], TOL[dtype])
    return got, ref, errs


def make_state(host, dtype):
    """Device-side module state for update_block / adamw: masters, moments, grads, working copies."""
    st = {}
    for name in ("A", "B"):
        master = host[name].to(torch.float32).cuda().contiguous()
        st[name] = dict(master=master, m=torch.zeros_like(master), v=torch.zeros_like(master),
                        grad=torch.zeros_like(master),
                        work=master.to(torch.bfloat16).contiguous() if dtype == "bf16" else None)
    return st


def snapshot_block(blk):
    """Host fp64 copies of everything the oracle needs from a runtime.Block, taken BEFORE the update."""
    projs = []
    for i, st in enumerate(blk.state):
        projs.append(dict(x=f64(blk.x[i]), dY=f64(blk.dY[i]), W0=f64(blk.W0[i]), s=blk.s,
                          A_master=f64(st["A"]["master"]), B_master=f64(st["B"]["master"]),
                          mA=f64(st["A"]["m"]), vA=f64(st["A"]["v"]), mB=f64(st["B"]["m"]), vB=f64(st["B"]["v"])))
    return projs


def step_bound(p0, ref, tol):
    """Tight bound on the optimizer's movement: tol * max|movement| plus one fp32 ulp of the parameter."""
    return tol * np.abs(ref - p0).max() + 2.0 ** -23 * np.abs(ref).max()


def ill_conditioned_mask(grad_log, i, nm, p0, hp, tol, m0=None, v0=None, step0=0, lrs=None):
    """Elements of projection i's A (or B) on which the optimizer's movement is ill-conditioned under the
    gradient's own tolerance: a gradient error of tol * max|g| in one of the steps (the most the gradient
    check lets through) moves the element by more than the tight bound.  Found by re-running the oracle's
    AdamW over the recorded per-step gradients with one step's gradient shifted by +-tol * max|g| at a time.
    For a single step from zero moments Adam's update is lr * g / (|g| + eps), sign-like, and the mask is
    exactly {|g| <= tol * max|g|}; over several steps it also holds the elements whose gradient changes
    sign or size between steps, where m_hat / sqrt(v_hat) is far from +-1.  Only there may the two sides
    legitimately take different steps."""
    gs = [(dA if nm == "A" else dB) for _, j, dA, dB in grad_log if j == i]
    assert gs, "no gradients recorded for this projection"
    n = len(gs)
    lrs = [hp["lr"]] * n if lrs is None else lrs
    m0 = np.zeros_like(p0) if m0 is None else m0
    v0 = np.zeros_like(p0) if v0 is None else v0

    def chain(grads):
        p, m, v = p0, m0, v0
        for k, g in enumerate(grads):
            p, m, v = orc.adamw_step(p, g, m, v, lrs[k], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"],
                                     step0 + k + 1)
        return p

    base = chain(gs)
    moved = np.zeros_like(p0)
    for k in range(n):
        shift = tol * np.abs(gs[k]).max()
        worst_k = np.zeros_like(p0)
        for sign in (1.0, -1.0):
            pert = list(gs)
            pert[k] = gs[k] + sign * shift
            worst_k = np.maximum(worst_k, np.abs(chain(pert) - base))
        moved += worst_k
    return moved > step_bound(p0, base, tol)


def check_adam_steps(name, p0, got, ref, small_g, tol, n_steps, lr, max_frac=0.02):
    """The optimizer's movement got - p0 against the oracle's ref - p0 (|movement| ~ n_steps * lr << |p|, so a check
    on p alone would pass a kernel that does nothing).  Tight bound: tol * max|movement| plus one fp32 ulp of p.
    Elements outside it must all be ones where the movement is ill-conditioned under the gradient tolerance
    (small_g, from ill_conditioned_mask), must stay within the worst case of a sign flip (2 lr per step), and
    must be few.  Returns their fraction."""
    assert np.isfinite(got).all(), f"{name}: non-finite master parameters"
    d_gpu, d_ref = got - p0, ref - p0
    assert np.abs(d_ref).max() > 0, f"{name}: the oracle did not move the parameters"
    bound = step_bound(p0, ref, tol)
    dev = np.abs(d_gpu - d_ref)
    off = dev > bound
    unexplained = off & ~small_g
    assert not unexplained.any(), (f"{name}: {int(unexplained.sum())} optimizer steps are off by up to "
                                   f"{dev[unexplained].max():.3e} (bound {bound:.3e}) where the step is well-conditioned")
    assert dev.max() <= 2.0 * n_steps * lr * (1.0 + 1e-3) + bound, f"{name}: a step is off by more than a sign flip"
    frac = float(off.mean())
    # (two elements are always allowed: on a tensor of a few hundred elements one element is already above 1e-3)
    assert frac <= max(max_frac, 2.0 / got.size), f"{name}: {frac:.4f} of the optimizer steps are off"
    return frac


def compare_block(blk, projs0, ref, epochs, hp, tol=1e-2, check_io=True, grad_log=None):
    """Device state of a block after templora_update_block against the oracle's update_block.  `epochs` is the
    number of optimizer steps taken (from zero moments, constant rate hp["lr"]); grad_log the per-step
    gradients recorded by the oracle."""
    lr = hp["lr"]
    worst = {}
    fracs = {}
    for i, (q, st) in enumerate(zip(ref, blk.state)):
        name = blk.names[i]
        if check_io:
            worst[f"{name}.y"] = assert_close(f"{name}.y", f64(blk.y[i]), q["y"], tol)
            if blk.dX[i] is not None:
                worst[f"{name}.dX"] = assert_close(f"{name}.dX", f64(blk.dX[i]), q["dX"], tol)
        worst[f"{name}.dA"] = assert_close(f"{name}.dA", f64(st["A"]["grad"]), q["dA"], tol)
        worst[f"{name}.dB"] = assert_close(f"{name}.dB", f64(st["B"]["grad"]), q["dB"], tol)
        for nm in ("A", "B"):
            p0 = projs0[i][nm + "_master"]
            got = f64(st[nm]["master"])
            fracs[f"{name}.{nm}"] = check_adam_steps(f"{name}.{nm}", p0, got, q[nm + "_master"],
                                                     ill_conditioned_mask(grad_log, i, nm, p0, hp, tol,
                                                                          m0=projs0[i].get("m" + nm),
                                                                          v0=projs0[i].get("v" + nm)),
                                                     tol, epochs, lr)
            assert_close(f"{name}.m{nm}", f64(st[nm]["m"]), q["m" + nm], tol)
            assert_close(f"{name}.v{nm}", f64(st[nm]["v"]), q["v" + nm], 2 * tol)
            assert np.array_equal(f64(st[nm]["work"]), orc.round_bf16(got.astype(np.float32))), f"{name}.{nm} work copy"
    print("fraction of optimizer steps outside the tight bound (all ill-conditioned under the gradient tolerance):",
          {k: f"{v:.4f}" for k, v in fracs.items()})
    return worst
