"""Calls the SiLU-gating and RMSNorm entry points twice on fresh bf16 tensors of 7B widths and exits.
A small, self-ending program to run under a profiler (run it from the repository root):

    python paper_2401_11504_b200/examples/block_ops_once.py
"""
import os
import sys

import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
from paper_2401_11504_b200 import binding as b  # noqa: E402


def main():
    dev, T = "cuda", 4096
    bf = dict(device=dev, dtype=torch.bfloat16)
    g = [torch.randn(T, 11008, **bf) for _ in range(2)]
    u = [torch.randn(T, 11008, **bf) for _ in range(2)]
    dh = [torch.randn(T, 11008, **bf) for _ in range(2)]
    o0, o1 = torch.empty_like(g[0]), torch.empty_like(g[0])
    x = [torch.randn(4 * T, 4096, **bf) for _ in range(2)]
    dy = [torch.randn(4 * T, 4096, **bf) for _ in range(2)]
    y, w = torch.empty_like(x[0]), torch.rand(4096, **bf)
    for i in range(2):
        b.templora_swiglu_fwd(g[i], u[i], o0)
        b.templora_swiglu_bwd(g[i], u[i], dh[i], o0, o1)
        b.templora_rmsnorm_fwd(x[i], w, 1e-5, y)
        b.templora_rmsnorm_bwd(x[i], w, dy[i], 1e-5, y)
    torch.cuda.synchronize()
    print("ok")


if __name__ == "__main__":
    main()
