"""LoRA dropout on the low-rank branch input (the paper's training setting, p = 0.05): the device's
Philox4x32-10 mask must equal the oracle's bit for bit, and forward, backward and the chunk update
with dropout must match the oracle within the usual tolerances."""
import numpy as np
import pytest
import torch

from oracle import templora_oracle as orc
from paper_2401_11504_b200 import inputs
from parity_utils import TOL, assert_close, check_fwd_bwd, f64, hp32, make_state

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2401_11504_b200 import build
    build.build_library()
    from paper_2401_11504_b200 import binding
    binding.templora_set_kernel_path(0)
    return binding


@pytest.mark.parametrize("dtype,T,d", [("bf16", 300, 64), ("bf16", 129, 128), ("f32", 50, 24)])
@pytest.mark.parametrize("p,seed,offset", [(0.05, 1234, 0), (0.5, (7 << 32) | 99, (3 << 32) | 5)])
def test_device_mask_equals_oracle_mask_bit_for_bit(b, dtype, T, d, p, seed, offset):
    # A = identity (exact in bf16) makes U = xd = x * keep / (1 - p): the saved U shows the mask
    td = torch.bfloat16 if dtype == "bf16" else torch.float32
    x = inputs.make_tensor(40, "mask", f"x{T}{d}", (T, d), "normal", 1.0, dtype).cuda()
    x = torch.where(x == 0, torch.ones_like(x), x)
    W0 = torch.zeros((d, d), dtype=td, device="cuda")
    A = torch.eye(d, dtype=td, device="cuda")
    B = torch.zeros((d, d), dtype=td, device="cuda")
    lin = b.linear_desc(W0, A, B, 1.0, dropout_p=p, dropout_seed=seed, dropout_offset=offset)
    ws = b.alloc_workspace(b.templora_workspace_bytes(lin, T))
    y = torch.empty((T, d), dtype=td, device="cuda")
    U = torch.full((T, d), float("nan"), dtype=torch.float32, device="cuda")
    b.templora_linear_fwd(lin, x, y, ws, U_save=U)
    assert b.templora_read_device_status(ws)[0] == 0
    p32 = float(np.float32(p))
    keep = orc.dropout_keep(seed, offset, T, d, p32)
    got_keep = (f64(U) != 0).astype(np.uint8)
    assert np.array_equal(got_keep, keep), f"{(got_keep != keep).sum()} mask bits differ"
    assert 0 < keep.sum() < keep.size
    want = f64(x) * keep / (1.0 - p32)
    assert_close("xd", f64(U), want, 1e-2 if dtype == "bf16" else 1e-6)


@pytest.mark.parametrize("T,d_in,d_out,r", [(300, 328, 520, 24), (640, 1024, 768, 64), (128, 512, 512, 128)])
@pytest.mark.parametrize("p", [0.05, 0.5])
def test_dropout_fwd_bwd_tensor_core_path(b, T, d_in, d_out, r, p):
    check_fwd_bwd(b, 41, f"drop-{T}-{d_in}-{d_out}-{r}-{p}", T, d_in, d_out, r, 2.0, "bf16", dropout=(p, 555, 17))


def test_dropout_without_saved_U_and_without_dX(b):
    check_fwd_bwd(b, 42, "drop-opts", 200, 256, 384, 64, 1.0, "bf16", dropout=(0.05, 1, 2), save_U=False, with_dX=False)


@pytest.mark.parametrize("dtype,T,d_in,d_out,r", [("f32", 128, 512, 512, 8), ("f32", 37, 100, 67, 5), ("bf16", 65, 100, 36, 5)])
def test_dropout_fwd_bwd_generic_path(b, dtype, T, d_in, d_out, r):
    check_fwd_bwd(b, 43, f"dropg-{dtype}-{T}", T, d_in, d_out, r, 2.0, dtype, dropout=(0.05, 99, 3))


def _update_with_dropout(b, dtype, shapes, T, r, epochs, batch, p, hp, seed):
    hp = hp32(hp)
    p32 = float(np.float32(p))
    hosts = [inputs.make_linear(seed, f"dub{i}", T, di, do, r, dtype=dtype) for i, (di, do) in enumerate(shapes)]
    devs = [{k: v.cuda() for k, v in h.items()} for h in hosts]
    states = [make_state(h, dtype) for h in hosts]
    lins, As, Bs, ys, dXs = [], [], [], [], []
    for i, (d, st) in enumerate(zip(devs, states)):
        a = st["A"]["work"] if dtype == "bf16" else st["A"]["master"]
        bb = st["B"]["work"] if dtype == "bf16" else st["B"]["master"]
        lins.append(b.linear_desc(d["W0"], a, bb, 2.0, dropout_p=p, dropout_seed=1000 + i, dropout_offset=10 * i))
        As.append(b.param_desc(st["A"]["master"], st["A"]["m"], st["A"]["v"], st["A"]["grad"], st["A"]["work"]))
        Bs.append(b.param_desc(st["B"]["master"], st["B"]["m"], st["B"]["v"], st["B"]["grad"], st["B"]["work"]))
        ys.append(torch.full_like(d["dY"], float("nan")))
        dXs.append(torch.full_like(d["x"], float("nan")))
    ws = b.alloc_workspace(b.templora_update_block_workspace_bytes(lins, T))
    args = b.UpdateBlockArgs(lins, As, Bs, [d["x"] for d in devs], [d["dY"] for d in devs], ys, dXs)
    step = b.templora_update_block_batched(args, batch, epochs, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
                                           hp["weight_decay"], 0, ws)
    assert b.templora_read_device_status(ws)[0] == 0
    projs = [dict(x=f64(h["x"]), dY=f64(h["dY"]), W0=f64(h["W0"]), s=2.0, A_master=f64(h["A"]), B_master=f64(h["B"]),
                  dropout_seed=1000 + i, dropout_offset=10 * i) for i, h in enumerate(hosts)]
    ref, rstep = orc.update_block(projs, epochs, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"],
                                  bf16_work=(dtype == "bf16"), batch=batch, dropout_p=p32)
    assert rstep == step == epochs * -(-T // batch)
    tol = TOL[dtype]
    for i, (q, st) in enumerate(zip(ref, states)):
        assert_close(f"y{i}", f64(ys[i]), q["y"], tol)
        assert_close(f"dX{i}", f64(dXs[i]), q["dX"], tol)
        assert_close(f"dA{i}", f64(st["A"]["grad"]), q["dA"], tol)
        assert_close(f"dB{i}", f64(st["B"]["grad"]), q["dB"], tol)
        assert_close(f"mA{i}", f64(st["A"]["m"]), q["mA"], tol)
        assert_close(f"mB{i}", f64(st["B"]["m"]), q["mB"], tol)
    # dropout is really on: the plain update gives a different first moment
    plain, _ = orc.update_block(projs, epochs, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"],
                                bf16_work=(dtype == "bf16"), batch=batch)
    assert np.abs(plain[0]["mA"] - ref[0]["mA"]).max() > 10 * tol * np.abs(ref[0]["mA"]).max()


def test_update_block_with_dropout_bf16(b):
    _update_with_dropout(b, "bf16", [(256, 384), (384, 256), (256, 256)], 400, 64, 2, 256, 0.25,
                         dict(lr=2e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0), 44)


def test_update_block_with_dropout_paper_setting(b):
    _update_with_dropout(b, "bf16", [(512, 512), (512, 1408)], 512, 64, 2, 512, 0.05, dict(inputs.ADAMW), 45)


def test_update_block_with_dropout_fp32(b):
    _update_with_dropout(b, "f32", [(96, 80)], 70, 8, 1, 32, 0.3,
                         dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0), 46)
