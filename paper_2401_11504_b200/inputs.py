"""Seeded synthetic inputs for the Temp-Lora chunk-update path.

This module only draws numbers and names shapes.  It holds none of the method's
arithmetic, imports neither the CUDA binding nor the oracle, and serves both
sides of every parity test, so the two see bit-identical tensors.

Distributions (one LoRA-augmented projection):
    x  ~ N(0, 1)                       [T, d_in]     activations of the chunk
    W0 ~ N(0, variance 1/d_in)         [d_out, d_in] frozen base weight
    A  ~ U(-1/sqrt(d_in), 1/sqrt(d_in))[r, d_in]
    B  ~ N(0, std 0.02)                [d_out, r]    (non-zero so that dA != 0)
    dY ~ N(0, 1)                       [T, d_out]    upstream gradient
These stand in for real activations of the models the paper evaluates
(Llama-2 7B/13B/70B-class projections, chunk sizes 1024..4096, rank 64):
GEMM/GEMV time does not depend on values, only on shapes.

Host tensors come from numpy's counter-based Philox generator keyed by
(seed, tag, tensor name), so any tensor can be regenerated alone.  Tensors made
directly on a CUDA device (full-size benchmark weights) use torch's device
generator seeded from the same key.  bf16 configurations round once, here, to
bfloat16 storage; both sides then read the same bf16 values.
"""
import hashlib
import math

import numpy as np
import torch

# (name, d_in, d_out) of the seven LoRA-carrying projections of one decoder block
LLAMA2_7B_BLOCK = [
    ("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
    ("gate", 4096, 11008), ("up", 4096, 11008), ("down", 11008, 4096),
]
LLAMA2_70B_BLOCK = [  # grouped-query attention: k, v project to 1024
    ("q", 8192, 8192), ("k", 8192, 1024), ("v", 8192, 1024), ("o", 8192, 8192),
    ("gate", 8192, 28672), ("up", 8192, 28672), ("down", 28672, 8192),
]

# other models the paper evaluates (Section "Experiments"): block shapes for the rank / chunk / batch sweeps
LLAMA2_13B_BLOCK = [
    ("q", 5120, 5120), ("k", 5120, 5120), ("v", 5120, 5120), ("o", 5120, 5120),
    ("gate", 5120, 13824), ("up", 5120, 13824), ("down", 13824, 5120),
]
MISTRAL_7B_BLOCK = [  # grouped-query attention, 8 kv heads
    ("q", 4096, 4096), ("k", 4096, 1024), ("v", 4096, 1024), ("o", 4096, 4096),
    ("gate", 4096, 14336), ("up", 4096, 14336), ("down", 14336, 4096),
]
YI_6B_BLOCK = [  # grouped-query attention, 4 kv heads
    ("q", 4096, 4096), ("k", 4096, 512), ("v", 4096, 512), ("o", 4096, 4096),
    ("gate", 4096, 11008), ("up", 4096, 11008), ("down", 11008, 4096),
]
BLOCKS = {"llama2_7b": LLAMA2_7B_BLOCK, "llama2_13b": LLAMA2_13B_BLOCK, "llama2_70b": LLAMA2_70B_BLOCK,
          "mistral_7b": MISTRAL_7B_BLOCK, "yi_6b": YI_6B_BLOCK}

ADAMW = dict(lr=5e-5, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0)

# The five workload configurations (index = configuration number).
CONFIGS = [
    dict(name="single_fp32", dtype="f32", T=128, r=8, s=2.0, projections=[("lin", 512, 512)],
         n_blocks=1, epochs=1),
    dict(name="llama2_7b_block", dtype="bf16", T=1024, r=64, s=2.0, projections=LLAMA2_7B_BLOCK,
         n_blocks=1, epochs=1),
    dict(name="llama2_7b_32blocks", dtype="bf16", T=1024, r=64, s=2.0, projections=LLAMA2_7B_BLOCK,
         n_blocks=32, epochs=2),
    dict(name="llama2_7b_decode", dtype="bf16", T=16, r=64, s=2.0, projections=LLAMA2_7B_BLOCK,
         n_blocks=32, epochs=0, decode_tokens=(1, 4, 16)),
    dict(name="llama2_70b_block", dtype="bf16", T=4096, r=64, s=2.0, projections=LLAMA2_70B_BLOCK,
         n_blocks=1, epochs=1),
]


def _key(seed, tag, name):
    h = hashlib.sha256(f"{int(seed)}|{tag}|{name}".encode()).digest()
    return int.from_bytes(h[:16], "little")


def _host_normal(key, shape, std):
    g = np.random.Generator(np.random.Philox(key=key))
    a = g.standard_normal(size=shape, dtype=np.float32)
    a *= np.float32(std)
    return a


def _host_uniform(key, shape, bound):
    g = np.random.Generator(np.random.Philox(key=key))
    a = g.random(size=shape, dtype=np.float32)
    a *= np.float32(2.0 * bound)
    a -= np.float32(bound)
    return a


def _torch_dtype(dtype):
    return {"f32": torch.float32, "bf16": torch.bfloat16}[dtype]


def make_tensor(seed, tag, name, shape, kind, scale, dtype="f32", device="cpu"):
    """One seeded tensor.  kind: 'normal' (scale = std) or 'uniform' (scale = bound)."""
    key = _key(seed, tag, name)
    td = _torch_dtype(dtype)
    dev = torch.device(device)
    if dev.type == "cpu":
        a = _host_normal(key, shape, scale) if kind == "normal" else _host_uniform(key, shape, scale)
        return torch.from_numpy(a).to(td)
    gen = torch.Generator(device=dev)
    gen.manual_seed(key & ((1 << 63) - 1))
    if kind == "normal":
        t = torch.randn(shape, generator=gen, device=dev, dtype=torch.float32) * scale
    else:
        t = (torch.rand(shape, generator=gen, device=dev, dtype=torch.float32) * 2.0 - 1.0) * scale
    return t.to(td)


def make_linear(seed, tag, T, d_in, d_out, r, dtype="f32", device="cpu", zero_B=False):
    """All tensors of one projection, in storage dtype `dtype`, keyed by name."""
    mk = lambda name, shape, kind, scale: make_tensor(seed, tag, name, shape, kind, scale, dtype, device)
    out = dict(
        x=mk("x", (T, d_in), "normal", 1.0),
        W0=mk("W0", (d_out, d_in), "normal", 1.0 / math.sqrt(d_in)),
        A=mk("A", (r, d_in), "uniform", 1.0 / math.sqrt(d_in)),
        B=mk("B", (d_out, r), "normal", 0.02),
        dY=mk("dY", (T, d_out), "normal", 1.0),
    )
    if zero_B:
        out["B"] = torch.zeros_like(out["B"])
    return out


def to_f64(t):
    """Exact widening of a stored tensor (fp32 or bf16) to a float64 numpy array."""
    return t.detach().to("cpu").to(torch.float64).numpy()


# ---- algorithmic work per unit (used by the benchmark's roofline arithmetic) ----
def flops_fwd_bwd(T, d_in, d_out, r):
    """Useful flops of forward + backward of one projection: the two frozen-weight
    GEMMs (4 T d_in d_out) and the six rank-r products (6 T r (d_in + d_out))."""
    return 4 * T * d_in * d_out + 6 * T * r * (d_in + d_out)


def adamw_bytes(n_params):
    """Read g, p, m, v (fp32) and write p, m, v (fp32) plus the bf16 working copy."""
    return 30 * n_params


def decode_bytes(d_in, d_out, r):
    """bf16 W0, A and B streamed once per decode step of one projection."""
    return 2 * d_in * d_out + 2 * r * (d_in + d_out)
