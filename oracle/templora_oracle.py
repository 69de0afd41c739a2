"""fp64 CPU oracle for the Temp-Lora chunk-update hot path.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA library is checked against.  It shares no code with the CUDA path and is
imported only by the tests, by the smoke check and by the CPU-baseline leg of
the benchmark.  The product never calls it.

What it computes (Temp-Lora, Section "Temp-Lora" and Algorithm 1, the training
step of the module Theta_k over a chunk; the module is the LoRA
module of Hu et al. that the paper adopts by citation, with the hyper-parameters
of the paper's "Setup" paragraph: alpha = 64, rank = 64, learning rate 5e-5,
n = 2 epochs, bfloat16 training):

    U  = x A^T                         [T, r]
    y  = x W0^T + s U B^T              [T, d_out]         s = alpha / r
    V  = dY B                          [T, r]
    dX = dY W0 + s V A                 [T, d_in]
    dB = s dY^T U                      [d_out, r]
    dA = s V^T x                       [r, d_in]
    (W0 is frozen: the method never alters the base model, so no dW0 exists.)

With LoRA dropout (paper's Setup: dropout = 0.05; in LoRA the dropout sits on the input of
the low-rank branch) the branch reads xd = x * keep / (1 - p) instead of x:
    U = xd A^T ;  dA = s V^T xd ;  dX = dY W0 + s (V A) * keep / (1 - p) ;  y, V, dB as above.
keep[t,k] in {0,1} comes from the counter-based generator Philox4x32-10 (Salmon, Moraes, Dror,
Shaw, "Parallel random numbers: as easy as 1, 2, 3", SC'11), written out below from its
published definition.

Every function is the definition written out with numpy matmuls on float64
arrays, in the order above; nothing is blocked, fused or reordered.

Pins (tests/test_oracle_pins.py): brute-force Python loops on tiny shapes, an
integer worked example under tests/golden/, B = 0 reduction, the merged-weight
identity, exact finite differences (the loss sum(dY*y) is linear in each of
x, A, B separately), additivity of dA/dB over row partitions, the closed-form
first AdamW step, the constant-gradient AdamW trajectory, and torch's own
bfloat16 cast for the rounding helper.  The dropout mask: the generator against
its published known-answer vectors, and the element -> (counter, word) layout
against a hand case built from the first of those vectors and against a scalar
restatement of the rule with 64-bit seeds and offsets and rows that start inside
a block.

Every function of this file has at least one such pin; none is left unpinned.
The paper itself prints no worked numeric example and no per-layer value for
this path, so no pin compares with a number printed there: the pins are what the
mathematics fixes (closed forms, brute force, exact finite differences, textbook
special cases, a published generator's known answers).
"""
import numpy as np

F64 = np.float64


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=F64))


# --------------------------------------------------------------------------
# forward:  y = x W0^T + s (x A^T) B^T            (Temp-Lora module forward)
# --------------------------------------------------------------------------
def linear_fwd(x, W0, A, B, s, keep=None, p=0.0):
    """x [T,d_in], W0 [d_out,d_in], A [r,d_in], B [d_out,r] -> (y [T,d_out], U [T,r]).
    keep [T,d_in] of 0/1 and p: LoRA dropout on the input of the low-rank branch."""
    x, W0, A, B = _f64(x), _f64(W0), _f64(A), _f64(B)
    xd = x if keep is None else x * _f64(keep) / (1.0 - F64(p))
    U = xd @ A.T
    y = x @ W0.T + F64(s) * (U @ B.T)
    return y, U


# --------------------------------------------------------------------------
# backward with W0 frozen (no dW0: the base model is never altered)
# --------------------------------------------------------------------------
def linear_bwd(x, dY, W0, A, B, s, keep=None, p=0.0):
    """-> (dX [T,d_in], dA [r,d_in], dB [d_out,r]); gradients are plain sums over tokens."""
    x, dY, W0, A, B = _f64(x), _f64(dY), _f64(W0), _f64(A), _f64(B)
    s = F64(s)
    scale = 1.0 if keep is None else _f64(keep) / (1.0 - F64(p))   # d xd / d x, elementwise
    xd = x * scale
    U = xd @ A.T
    V = dY @ B
    dX = dY @ W0 + s * (V @ A) * scale
    dB = s * (dY.T @ U)
    dA = s * (V.T @ xd)
    return dX, dA, dB


# --------------------------------------------------------------------------
# Philox4x32-10 and the dropout mask drawn from it
# --------------------------------------------------------------------------
_PHILOX_M0, _PHILOX_M1 = np.uint64(0xD2511F53), np.uint64(0xCD9E8D57)
_PHILOX_W0, _PHILOX_W1 = np.uint64(0x9E3779B9), np.uint64(0xBB67AE85)
_MASK32 = np.uint64(0xFFFFFFFF)


def philox4x32_10(counter, key):
    """counter: uint32 array [..., 4], key: (k0, k1).  Ten rounds of
        (c0, c1, c2, c3) <- (hi(M1*c2) ^ c1 ^ k0,  lo(M1*c2),  hi(M0*c0) ^ c3 ^ k1,  lo(M0*c0))
    with the key bumped by the Weyl constants after every round.  Returns uint32 [..., 4]."""
    c = np.asarray(counter, dtype=np.uint64)
    c0, c1, c2, c3 = c[..., 0], c[..., 1], c[..., 2], c[..., 3]
    k0, k1 = np.uint64(int(key[0]) & 0xFFFFFFFF), np.uint64(int(key[1]) & 0xFFFFFFFF)
    for _ in range(10):
        p0, p1 = _PHILOX_M0 * c0, _PHILOX_M1 * c2          # 32 x 32 -> 64 bit products
        c0, c1, c2, c3 = ((p1 >> np.uint64(32)) ^ c1 ^ k0, p1 & _MASK32,
                          (p0 >> np.uint64(32)) ^ c3 ^ k1, p0 & _MASK32)
        k0, k1 = (k0 + _PHILOX_W0) & _MASK32, (k1 + _PHILOX_W1) & _MASK32
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def dropout_threshold(p):
    """An element is dropped iff its 32-bit draw is below floor(p * 2^32)."""
    return int(np.floor(float(p) * 4294967296.0))


def dropout_keep(seed, offset, T, d_in, p):
    """keep [T, d_in] of 0/1.  Element e = t*d_in + k takes word e % 4 of
    Philox4x32-10(counter = (lo(e/4), hi(e/4), lo(offset), hi(offset)), key = (lo(seed), hi(seed)))."""
    n = int(T) * int(d_in)
    q = np.arange((n + 3) // 4, dtype=np.uint64)
    ctr = np.empty((q.size, 4), dtype=np.uint64)
    ctr[:, 0], ctr[:, 1] = q & _MASK32, q >> np.uint64(32)
    ctr[:, 2], ctr[:, 3] = np.uint64(int(offset) & 0xFFFFFFFF), np.uint64((int(offset) >> 32) & 0xFFFFFFFF)
    draws = philox4x32_10(ctr, (int(seed) & 0xFFFFFFFF, (int(seed) >> 32) & 0xFFFFFFFF)).reshape(-1)[:n]
    return (draws >= np.uint32(min(dropout_threshold(p), 0xFFFFFFFF))).astype(np.uint8).reshape(int(T), int(d_in))


# --------------------------------------------------------------------------
# decode-time forward with the current module, token by token
# (Algorithm 1, generation step  Y[i] = Theta_k(...))
# --------------------------------------------------------------------------
def decode_fwd(x, W0, A, B, s):
    """x [n,d_in] (n generated-token rows) -> y [n,d_out]; one GEMV chain per token."""
    x, W0, A, B = _f64(x), _f64(W0), _f64(A), _f64(B)
    y = np.empty((x.shape[0], W0.shape[0]), dtype=F64)
    for i in range(x.shape[0]):
        u = A @ x[i]
        y[i] = W0 @ x[i] + F64(s) * (B @ u)
    return y


# --------------------------------------------------------------------------
# AdamW (decoupled weight decay, bias-corrected), step index t is 1-based
# --------------------------------------------------------------------------
def adamw_step(p, g, m, v, lr, beta1, beta2, eps, weight_decay, t):
    """Returns new (p, m, v).  eps is added to sqrt(v_hat), outside the root."""
    p, g, m, v = _f64(p), _f64(g), _f64(m), _f64(v)
    lr, beta1, beta2, eps, wd = F64(lr), F64(beta1), F64(beta2), F64(eps), F64(weight_decay)
    p = p * (1.0 - lr * wd)
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    m_hat = m / (1.0 - beta1 ** int(t))
    v_hat = v / (1.0 - beta2 ** int(t))
    p = p - lr * m_hat / (np.sqrt(v_hat) + eps)
    return p, m, v


# --------------------------------------------------------------------------
# bfloat16 storage rounding (round to nearest, ties to even) of fp32 values
# --------------------------------------------------------------------------
def round_bf16(a):
    """Value of `a` after fp32 -> bfloat16 storage (RNE), returned as float64."""
    f = np.ascontiguousarray(np.asarray(a, dtype=np.float32))
    bits = f.view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    rounded = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    out = rounded.astype(np.uint32).view(np.float32)
    out = np.where(np.isnan(f), f, out)
    return out.astype(F64)


# --------------------------------------------------------------------------
# the whole update of one block of projections: n epochs over the chunk,
# one optimizer step per epoch (batch = chunk)
# --------------------------------------------------------------------------
def lr_at_step(lr, step, warmup_steps):
    """Linear learning-rate warm-up ("Setup": the rate is warmed up linearly over the first two
    chunks): optimizer step `step` (1-based, counted over the whole run) uses
    lr * min(1, step / warmup_steps); warmup_steps <= 0 means a constant rate.  With E epochs and
    chunk/batch optimizer steps per epoch the paper's two chunks are warmup_steps = 2 * E * chunk/batch."""
    if warmup_steps is None or warmup_steps <= 0:
        return float(lr)
    return float(lr) * min(1.0, float(step) / float(warmup_steps))


def update_block(projs, epochs, lr, beta1, beta2, eps, weight_decay, step0=0, bf16_work=False, batch=None,
                 dropout_p=0.0, warmup_steps=0, lr_round=None, grad_log=None):
    """projs: list of dicts with keys x, dY, W0, s, A_master, B_master and optionally
    mA, vA, mB, vB (default 0).  For each epoch: forward and backward of every
    projection with the current working A, B; then step += 1 and AdamW on every
    A and B.  With bf16_work the GEMMs read round_bf16(master), the optimizer
    updates the master (fp32 master + bf16 working copy, which is what bfloat16
    training under ZeRO-2 implies).  With batch < T every epoch walks the chunk in
    row slices of `batch` tokens and takes one optimizer step per slice (the cost
    table's "training steps" = epochs * chunk / batch); y and dX are then filled
    slice by slice and dA, dB are the last slice's.  With dropout_p > 0 every optimizer step
    draws a fresh mask for its row slice: projection i uses seed projs[i]["dropout_seed"]
    and offset projs[i].get("dropout_offset", 0) + (number of steps taken before this one).

    A projection with key "dX_to" = j (an earlier projection with the same input width, typically q for k
    and v, gate for up: projections that read the same input) adds its input gradient into projection
    j's dX instead of keeping its own: state[j]["dX"] is then the gradient of the loss with respect to
    the shared input, and state[i]["dX"] is that same array.

    With warmup_steps > 0 the step numbered k (step0 + 1, step0 + 2, ...) uses lr_at_step(lr, k,
    warmup_steps); lr_round, if given, is applied to that rate (the tests pass the fp32 rounding
    that the C ABI's float argument imposes).

    grad_log, if a list, receives one entry (step, projection index, dA, dB) per projection and optimizer
    step: the gradients that step's AdamW consumed (a record for the tests; it changes nothing computed).

    Returns (state, step): state[i] has A_master, B_master, mA, vA, mB, vB and the
    last epoch's y, dX, dA, dB.
    """
    st = []
    for p in projs:
        A = _f64(p["A_master"])
        B = _f64(p["B_master"])
        st.append(dict(A_master=A, B_master=B,
                       mA=_f64(p.get("mA", np.zeros_like(A))), vA=_f64(p.get("vA", np.zeros_like(A))),
                       mB=_f64(p.get("mB", np.zeros_like(B))), vB=_f64(p.get("vB", np.zeros_like(B)))))
    step = int(step0)
    T = np.asarray(projs[0]["x"]).shape[0]
    batch = T if batch is None or batch >= T else int(batch)
    for p, q in zip(projs, st):
        q["y"] = np.zeros((T, np.asarray(p["W0"]).shape[0]), dtype=F64)
        q["dX"] = np.zeros((T, np.asarray(p["W0"]).shape[1]), dtype=F64)
    for _ in range(int(epochs)):
        for r0 in range(0, T, batch):
            rows = slice(r0, min(r0 + batch, T))
            for p, q in zip(projs, st):
                A = round_bf16(q["A_master"]) if bf16_work else q["A_master"]
                B = round_bf16(q["B_master"]) if bf16_work else q["B_master"]
                xb, dYb = _f64(p["x"])[rows], _f64(p["dY"])[rows]
                keep = None
                if dropout_p > 0:
                    keep = dropout_keep(p["dropout_seed"], p.get("dropout_offset", 0) + step, xb.shape[0],
                                        xb.shape[1], dropout_p)
                q["y"][rows], _ = linear_fwd(xb, p["W0"], A, B, p["s"], keep, dropout_p)
                dXb, q["dA"], q["dB"] = linear_bwd(xb, dYb, p["W0"], A, B, p["s"], keep, dropout_p)
                if p.get("dX_to") is None:
                    q["dX"][rows] = dXb
                else:
                    st[p["dX_to"]]["dX"][rows] += dXb
            step += 1
            if grad_log is not None:
                grad_log.extend((step, i, q["dA"].copy(), q["dB"].copy()) for i, q in enumerate(st))
            lr_k = lr_at_step(lr, step, warmup_steps)
            if lr_round is not None:
                lr_k = lr_round(lr_k)
            for q in st:
                q["A_master"], q["mA"], q["vA"] = adamw_step(q["A_master"], q["dA"], q["mA"], q["vA"],
                                                             lr_k, beta1, beta2, eps, weight_decay, step)
                q["B_master"], q["mB"], q["vB"] = adamw_step(q["B_master"], q["dB"], q["mB"], q["vB"],
                                                             lr_k, beta1, beta2, eps, weight_decay, step)
    for p, q in zip(projs, st):
        if p.get("dX_to") is not None:
            q["dX"] = st[p["dX_to"]]["dX"]
    return st, step


# ---------------------------------------------------------------------------
# The steps on either side of the projections inside a decoder block's update
# (the training step of Theta_k, Algorithm 1, runs a whole Llama-style block: RMSNorm -> q,k,v ... and
# gate, up -> SiLU(gate) * up -> down).  Plain definitions, fp64.
# ---------------------------------------------------------------------------
def swiglu_fwd(gate, up):
    """h = SiLU(gate) * up with SiLU(g) = g * sigmoid(g) (the Llama MLP's gating)."""
    g, u = _f64(gate), _f64(up)
    return g / (1.0 + np.exp(-g)) * u


def swiglu_bwd(gate, up, dh):
    """Gradients of h = SiLU(gate) * up:  dgate = dh * up * SiLU'(gate),  dup = dh * SiLU(gate),
    with SiLU'(g) = sigmoid(g) * (1 + g * (1 - sigmoid(g)))."""
    g, u, d = _f64(gate), _f64(up), _f64(dh)
    sg = 1.0 / (1.0 + np.exp(-g))
    return d * u * sg * (1.0 + g * (1.0 - sg)), d * g * sg


def rmsnorm_fwd(x, w, eps):
    """y[t, j] = x[t, j] / sqrt(mean_j x[t, j]^2 + eps) * w[j]  (Llama's RMSNorm; w is frozen here)."""
    x, w = _f64(x), _f64(w)
    rstd = 1.0 / np.sqrt(np.mean(x * x, axis=1, keepdims=True) + eps)
    return x * rstd * w


def rmsnorm_bwd(x, w, dy, eps):
    """dx of y = rmsnorm(x):  with xh = x * rstd and g = w * dy,
    dx = rstd * (g - xh * mean_j(xh * g)).  No weight gradient: the norm weights are not trained."""
    x, w, dy = _f64(x), _f64(w), _f64(dy)
    rstd = 1.0 / np.sqrt(np.mean(x * x, axis=1, keepdims=True) + eps)
    xh, g = x * rstd, w * dy
    return rstd * (g - xh * np.mean(xh * g, axis=1, keepdims=True))
