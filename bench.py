#!/usr/bin/env python
"""Benchmark of the Temp-Lora chunk update on B200.

    python bench.py --gpus N --steps K --warmup W [--impl reference]

A step is one pass of the whole hot path over one chunk: forward and backward of the seven
LoRA-augmented projections of a Llama-2-7B-shaped decoder block over T = 1024 tokens (rank 64,
s = 2) followed by one AdamW step on every A and B, through templora_update_block.  Steps rotate
over several blocks with distinct weights (each block's frozen weights alone are 405 MB, above the
126 MB L2).  N > 1 runs N independent replicas (the path does not shard), one process per GPU.

Prints one JSON line: the metric (chunk-update tokens/s), the end-to-end figure with host buffers,
the live roofline of the dominant kernel, the fp64 oracle timed on the host cores, clocks, and the
decode-time GEMV bandwidth.
"""
import argparse
import hashlib
import json
import os
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "temp_lora_chunk_update_tokens_per_s"
UNIT = "tokens/s"
WORKLOAD = "llama2_7b_block: 7 LoRA projections (q,k,v,o 4096x4096; gate,up 4096->11008; down 11008->4096), T=1024, r=64, s=2.0, fwd+bwd+AdamW, 1 epoch"
N_ROTATE = 4            # distinct blocks the timed steps rotate over
FALLBACK_PEAK_TFLOPS = 1400.0   # cuBLAS bf16, seconds-long loop under the power cap (used when no measured file exists)
FALLBACK_BURST_TFLOPS = 1590.0  # cuBLAS bf16, best of a short burst
FALLBACK_HBM_GBS = 6650.0
NOMINAL_TFLOPS = 2250.0         # dense bf16, data sheet

# DRAM traffic of one launch of the dominant kernel (bytes), from an ncu capture summarised under
# profiles/; valid only while the kernel source is the one that was profiled.
SHARED_INPUTS = [["q", "k", "v"], ["gate", "up"]]   # projections of a decoder block that read the same tensor
TRAFFIC = {"tc_gemm_sha1": "1fca5db76d4c8575304b020d1997996562109ab8", "bytes_per_launch": 1141020928}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return dict(tflops=float(p["bf16_tflops_sustained"]), burst=float(p["bf16_tflops"]), hbm=float(p["hbm_gbs"]),
                    source="measured")
    except Exception:
        return dict(tflops=FALLBACK_PEAK_TFLOPS, burst=FALLBACK_BURST_TFLOPS, hbm=FALLBACK_HBM_GBS, source="fallback")


def pick_regime(seconds, clocks):
    """Which measured cuBLAS figure a tensor-core number of this run is compared with.  The sustained
    figure was taken in a seconds-long loop with the SM clock pulled down by the power cap; it applies
    only when this run's timed region was also seconds long AND its sampled median SM clock sat below
    the maximum with the power cap active.  Everything else (short regions at full clock) is the burst regime."""
    mhz, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    capped = bool(mhz and mx and mhz < 0.95 * mx and "sw_power_cap" in (clocks.get("reasons") or []))
    return "sustained" if (seconds >= 2.0 and capped) else "burst"


def fractions(tflops, peaks, regime):
    """A tensor-core throughput against all three denominators, and the one that applies to this run."""
    if not tflops:
        return {"frac": None, "frac_of_burst": None, "frac_of_sustained": None, "frac_of_nominal_2250": None}
    out = {"frac_of_burst": tflops / peaks["burst"], "frac_of_sustained": tflops / peaks["tflops"],
           "frac_of_nominal_2250": tflops / NOMINAL_TFLOPS}
    out["frac"] = out["frac_of_sustained"] if regime == "sustained" else out["frac_of_burst"]
    return out


def kernel_sha1():
    """Fingerprint of the dominant kernel's source: tc_gemm.cu and the instruction wrappers it is written with."""
    h = hashlib.sha1()
    for name in ("tc_gemm.cu", "tc_device.cuh"):
        with open(os.path.join(ROOT, "paper_2401_11504_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def main_kernel_flops(projections, T, r):
    """Algorithmic flops of one launch of the fused GEMM kernel: y = x W0^T + s U B^T and
    dX = dY W0 + s V A for every projection (2 T d_in d_out each, plus the two rank-r products)."""
    return sum(4 * T * di * do + 2 * T * r * (di + do) for _, di, do in projections)


def block_flops(projections, T, r):
    from paper_2401_11504_b200 import inputs
    return sum(inputs.flops_fwd_bwd(T, di, do, r) for _, di, do in projections)


# ------------------------------------------------------------------ the oracle on the host cores
def oracle_sample_setup(seed, rows):
    """Host-side fp64 copies of one 7B-shaped block restricted to the first `rows` chunk tokens."""
    import numpy as np
    from paper_2401_11504_b200 import inputs
    c = inputs.CONFIGS[1]
    projs = []
    for name, d_in, d_out in c["projections"]:
        h = inputs.make_linear(seed, f"cpu/{name}", rows, d_in, d_out, c["r"], dtype="bf16")
        projs.append(dict(x=inputs.to_f64(h["x"]), dY=inputs.to_f64(h["dY"]), W0=inputs.to_f64(h["W0"]), s=c["s"],
                          A_master=inputs.to_f64(h["A"]), B_master=inputs.to_f64(h["B"])))
    return projs


def oracle_step(projs):
    from oracle import templora_oracle as orc
    from paper_2401_11504_b200 import inputs
    hp = inputs.ADAMW
    orc.update_block(projs, 1, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"], bf16_work=True)


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


ORACLE_ROWS = 1024      # the oracle's sample in BOTH legs below: the whole chunk (about a second per step on 16 cores)
ORACLE_SAMPLE = (f"all {ORACLE_ROWS} chunk tokens through all 7 projections of one 7B-shaped block "
                 "(fwd+bwd+AdamW, fp64 numpy oracle as it stands)")


def bench_config(parallelism):
    """The `config` object, identical in both arms: it names the workload and nothing run-dependent."""
    return {"workload": WORKLOAD,
            "l2": f"steps rotate over {N_ROTATE} blocks with distinct weights; each block's frozen weights alone exceed the 126 MB L2",
            "parallelism": parallelism}


def cpu_baseline(steps=8):
    """The oracle, as it stands, on the host cores: `steps` chunk updates of the whole sample after one warm-up."""
    projs = oracle_sample_setup(0, ORACLE_ROWS)
    oracle_step(projs)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(projs)
    dt = time.perf_counter() - t0
    return {"value": ORACLE_ROWS * steps / dt, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"{ORACLE_SAMPLE}; {steps} steps in {dt:.1f} s"}


def run_reference(args):
    """Reference arm: the fp64 oracle timed on the host cores, the same sample as the cpu_baseline leg."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    projs = oracle_sample_setup(0, ORACLE_ROWS)
    for _ in range(args.warmup):
        oracle_step(projs)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(projs)
    dt = time.perf_counter() - t0
    value = ORACLE_ROWS * args.steps / dt
    cores = blas_threads()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * dt / max(args.steps, 1), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": bench_config("replicas only" if args.gpus > 1 else "single GPU"),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{ORACLE_SAMPLE}; {args.steps} steps in {dt:.1f} s"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------ the CUDA arm
def run_ours(args):
    import torch
    from paper_2401_11504_b200 import build, inputs, runtime

    ranks = runtime.Ranks()
    if ranks.rank == 0:
        build.build_library()
    ranks.barrier()
    from paper_2401_11504_b200 import binding as b

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    torch.cuda.set_device(ranks.local_rank)
    dev = torch.device("cuda", ranks.local_rank)
    c = inputs.CONFIGS[1]
    T, r, s, projections = args.chunk, args.rank, c["s"], inputs.BLOCKS[args.model]
    batch = args.batch if args.batch else T
    default_workload = (args.model == "llama2_7b" and T == c["T"] and r == c["r"] and batch == T and args.epochs == 1
                        and args.dropout == 0.0 and not args.shared_input)
    workload = WORKLOAD if default_workload else (
        f"{args.model}_block: 7 LoRA projections, T={T}, batch={batch}, r={r}, s={s}, fwd+bwd+AdamW, {args.epochs} epoch(s), LoRA dropout {args.dropout}"
        + (", q,k,v and gate,up on shared inputs with summed dX" if args.shared_input else ""))
    hp = {k: float(v) for k, v in inputs.ADAMW.items()}
    peaks = load_peaks()

    stacked = args.stacked_blocks
    if stacked > 1:
        # the whole chunk update of a stack of blocks in ONE call (32 x 7 projections for the 7B stack):
        # distinct weights per block, x / dY / y / dX shared by the blocks per projection type
        default_workload = False
        workload = (f"{args.model}: {stacked} stacked blocks x 7 LoRA projections in one templora_update_block call, "
                    f"T={T}, batch={batch}, r={r}, s={s}, {args.epochs} epoch(s), LoRA dropout {args.dropout}")
        shared, stack = None, []
        for i in range(stacked):
            blk = runtime.Block(b, 0, f"r{ranks.rank}/stack{i}", projections, T, r, s, "bf16", dev, shared_io=shared,
                                dropout_p=args.dropout)
            shared = shared or blk.io
            stack.append(blk)
        cat = lambda f: [t for blk in stack for t in f(blk)]
        stack_args = b.UpdateBlockArgs(cat(lambda k: k.lins), cat(lambda k: k.A_desc), cat(lambda k: k.B_desc),
                                       cat(lambda k: k.x), cat(lambda k: k.dY), cat(lambda k: k.y), cat(lambda k: k.dX))
        blocks = stack
        update_args = [stack_args]
    else:
        blocks = [runtime.Block(b, 0, f"r{ranks.rank}/blk{i}", projections, T, r, s, "bf16", dev, dropout_p=args.dropout,
                                input_groups=SHARED_INPUTS if args.shared_input else None)
                  for i in range(args.blocks)]
        update_args = [blk.args for blk in blocks]
    N_ROT = len(update_args)
    ws_need = b.templora_update_block_workspace_bytes(blocks[0].lins, T)
    if stacked > 1:
        ws_need = max(ws_need, b.templora_update_block_workspace_bytes(cat(lambda k: k.lins), T))
    ws = b.alloc_workspace(ws_need, dev)
    steps_taken = [0] * N_ROT

    def step(i):
        k = i % N_ROT
        steps_taken[k] = b.templora_update_block_batched(update_args[k], batch, args.epochs, hp["lr"], hp["beta1"],
                                                         hp["beta2"], hp["eps"], hp["weight_decay"], steps_taken[k], ws)

    for i in range(max(args.warmup, 3)):
        step(i)
    torch.cuda.synchronize()
    for k in range(b.N_KINDS):
        b.templora_timing_read(k, reset=True)

    # ---- timed region: inputs resident in HBM --------------------------------
    stream = torch.cuda.current_stream()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    b.templora_timing_enable([b.KIND_TC_MAIN])   # events around the dominant kernel only
    ranks.barrier()
    torch.cuda.synchronize()
    with runtime.ClockSampler(torch.cuda.current_device()) as clk:
        ev0.record(stream)
        for i in range(args.steps):
            step(i)
        ev1.record(stream)
        torch.cuda.synchronize()
    ranks.barrier()
    b.templora_timing_enable(False)
    seconds = ev0.elapsed_time(ev1) / 1e3
    code, where = b.templora_read_device_status(ws)
    assert code == 0, f"device status {code} at {where}"

    launches = 0
    per_kind = {}
    for k in range(b.N_KINDS):
        ms, timed, allc = b.templora_timing_read(k, reset=True)
        per_kind[k] = (ms, timed, allc)
        launches += allc
    value, slowest = runtime.aggregate_throughput(T * args.steps, seconds, ranks)

    # ---- roofline of the dominant kernel (fused GEMM, 256-wide tiles), measured live ----
    ms_main, n_main, _ = per_kind[b.KIND_TC_MAIN]
    # one launch of the fused kernel covers one batch of rows of every projection
    launches_per_step = args.epochs * -(-T // batch)
    flops_main = main_kernel_flops(projections, T, r) * args.epochs / launches_per_step
    if args.dropout > 0:   # the rank-r term of dX runs in its own masked pass then
        flops_main -= sum(2 * T * r * di for _, di, _ in projections) * args.epochs / launches_per_step
    if stacked > 1:
        # groups of 8 projections straddle the blocks: average over all launches of a step instead
        total = flops_main * launches_per_step * stacked * args.steps
        flops_main = total / max(n_main, 1)
    achieved = flops_main / (ms_main / n_main * 1e-3) / 1e12 if n_main else None
    clocks = clk.summary()
    regime = pick_regime(seconds, clocks)
    sha = kernel_sha1()
    traffic = TRAFFIC["bytes_per_launch"] if (TRAFFIC["tc_gemm_sha1"] == sha and default_workload) else None
    roofline = {"bound": "tensor", "kernel": "pair::tc_gemm_pair_kernel (y and dX of every projection of the block, rank-r terms fused)",
                "achieved": achieved, "peak": peaks["tflops"] if regime == "sustained" else peaks["burst"],
                "unit": "TFLOP/s", **fractions(achieved, peaks, regime), "traffic": traffic,
                "regime": regime,
                "peak_source": (f"{peaks['source']}: cuBLAS bf16 8192^3, burst {peaks['burst']} / sustained {peaks['tflops']} TFLOP/s; "
                                f"this run: timed region {seconds:.3f} s, median SM clock {clocks.get('sm_mhz')} of "
                                f"{clocks.get('sm_max_mhz')} MHz, reasons {clocks.get('reasons')} -> {regime} figure applies"),
                "algorithmic_flops_per_launch": flops_main,
                "launch_ms": ms_main / n_main if n_main else None, "launches_timed": n_main}
    # the same frozen-weight products through cuBLAS (torch.matmul: no LoRA terms, 14 separate launches),
    # timed right here in the same clock regime: context for the fraction above, not a denominator
    if default_workload and ranks.world == 1:
        roofline["cublas_same_shapes_tflops"] = cublas_same_shapes(torch, blocks, projections, T, min(args.steps, 50))
    # shares of the other kernels: a separate short pass with events around every launch
    for k in range(b.N_KINDS):
        b.templora_timing_read(k, reset=True)
    b.templora_timing_enable(True)
    e0s, e1s = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_share = min(args.steps, 20)
    e0s.record(stream)
    for i in range(n_share):
        step(i)
    e1s.record(stream)
    torch.cuda.synchronize()
    b.templora_timing_enable(False)
    share_ms = e0s.elapsed_time(e1s)
    kernel_share = {}
    for name, k in (("tc_main", b.KIND_TC_MAIN), ("tc_skinny", b.KIND_TC_SKINNY), ("reduce", b.KIND_REDUCE),
                    ("adamw", b.KIND_ADAMW), ("dropout", b.KIND_DROPOUT), ("tc_dropout_term", b.KIND_TC_DROPOUT_TERM)):
        ms, _, _ = b.templora_timing_read(k, reset=True)
        kernel_share[name] = round(ms / max(share_ms, 1e-9), 4)

    # ---- end to end: host buffers in, updated module out, copies inside the timed region ----
    # Every step copies that step's x and dY from pinned host memory to the device, runs the chunk
    # update and copies the updated bf16 A and B back.  The device input buffers are double-buffered:
    # the copy of step i+1 runs on a second stream while step i computes (what a serving loop does).
    blk = blocks[0]
    ins0 = blk.x + blk.dY
    ins1 = [torch.empty_like(t) for t in ins0]
    n_x = len(blk.x)
    args_e2e = [blk.args, b.UpdateBlockArgs(blk.lins, blk.A_desc, blk.B_desc, ins1[:n_x], ins1[n_x:], blk.y, blk.dX)]
    dev_in = [ins0, ins1]
    host_in = [torch.empty_like(t, device="cpu").pin_memory().copy_(t) for t in ins0]
    outs = [st[nm]["work"] for st in blk.state for nm in ("A", "B")]
    host_out = [torch.empty_like(t, device="cpu").pin_memory() for t in outs]
    h2d = sum(h.numel() * h.element_size() for h in host_in)
    d2h = sum(h.numel() * h.element_size() for h in host_out)
    copy_stream = torch.cuda.Stream(device=dev)
    ready = [torch.cuda.Event(), torch.cuda.Event()]     # inputs of buffer set k have landed
    consumed = [torch.cuda.Event(), torch.cuda.Event()]  # the update that read buffer set k is done

    def upload(i):
        k = i % 2
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(consumed[k])
            for h, d in zip(host_in, dev_in[k]):
                d.copy_(h, non_blocking=True)
            ready[k].record(copy_stream)

    def e2e_run(n_steps):
        for k in range(2):
            consumed[k].record(stream)
        upload(0)
        for i in range(n_steps):
            k = i % 2
            if i + 1 < n_steps:
                upload(i + 1)
            stream.wait_event(ready[k])
            steps_taken[0] = b.templora_update_block_batched(args_e2e[k], batch, args.epochs, hp["lr"], hp["beta1"],
                                                             hp["beta2"], hp["eps"], hp["weight_decay"],
                                                             steps_taken[0], ws)
            consumed[k].record(stream)
            for h, d in zip(host_out, outs):
                h.copy_(d, non_blocking=True)
        torch.cuda.synchronize()

    e2e_run(3)
    n_e2e = max(3, min(args.steps, 30))
    ranks.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    e2e_run(n_e2e)
    e2e_seconds = time.perf_counter() - t0     # host clock around fully synchronised work: covers both streams
    e2e_seconds = ranks.max_over_ranks(e2e_seconds)
    e2e_value = ranks.sum_over_ranks(T * n_e2e) / e2e_seconds

    # ---- decode-time LoRA GEMV bandwidth (second figure of the metric) -------
    decode = None
    if not args.no_decode:
        decode = decode_bandwidth(b, torch, inputs, dev, peaks, n_blocks=args.decode_blocks)

    # ---- SiLU gating and RMSNorm (the element-wise steps of a block update beside the projections) ----
    block_ops = None
    if not args.no_decode:
        block_ops = block_ops_bandwidth(b, torch, inputs, dev, peaks)

    # ---- parallelized deployment: the update on one stream, decode on another, SMs split ----
    parallel = None
    if not args.no_parallel and default_workload and stacked <= 1:
        parallel = parallel_deployment(b, torch, runtime, blocks[0], hp)

    # ---- the other chunk-update configurations: 32 stacked blocks x 2 epochs in one call; the 70B block ----
    extra = {}
    if ranks.world == 1 and default_workload and not args.no_configs:
        del blocks, update_args, blk, args_e2e, dev_in, ins0, ins1, outs, ws
        torch.cuda.empty_cache()
        extra["config2"] = config_stack32(b, torch, inputs, runtime, dev, peaks, hp)
        torch.cuda.empty_cache()
        extra["config4"] = config_70b(b, torch, inputs, runtime, dev, peaks, hp)
        torch.cuda.empty_cache()
        extra["mlp"] = mlp_update(b, torch, inputs, runtime, dev, peaks, hp)
        torch.cuda.empty_cache()

    cpu = None
    if ranks.world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline()

    if ranks.rank == 0:
        tf_block = block_flops(projections, T, r) * args.epochs * max(stacked, 1) * args.steps / slowest / 1e12
        per_gpu = tf_block / ranks.world
        config = bench_config("replicas only" if ranks.world > 1 else "single GPU")
        if not default_workload:
            config["workload"] = workload
            config["l2"] = f"steps rotate over {N_ROT} blocks with distinct weights; each block's frozen weights alone exceed the 126 MB L2"
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": ranks.world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": 1e3 * slowest / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": config,
                "step": {"tflops": tf_block, "regime": regime,
                         **{k.replace("frac", "step_frac"): v for k, v in fractions(per_gpu, peaks, regime).items()}},
                "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                        "steps": n_e2e, "what": "per step: x and dY of the 7 projections from pinned host memory in (double-buffered, copy of step i+1 overlaps compute of step i), updated bf16 A and B out"},
                "gpu_launches": int(launches), "roofline": roofline, "kernel_time_share": kernel_share,
                "clocks": clocks, "cpu_baseline": cpu, "decode": decode, "block_ops": block_ops,
                "parallel_deployment": parallel, **extra}
        print(json.dumps(line))
    ranks.close()
    return 0


def run_only(args):
    """One of the side measurements alone, on cuda:0 (what the ncu captures under profiles/ run)."""
    import torch
    from paper_2401_11504_b200 import build, inputs, runtime
    build.build_library()
    from paper_2401_11504_b200 import binding as b
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = load_peaks()
    hp = {k: float(v) for k, v in inputs.ADAMW.items()}
    if args.only == "block_ops":
        out = block_ops_bandwidth(b, torch, inputs, dev, peaks, reps=1 if args.steps is None else args.steps)
    elif args.only == "mlp":
        out = mlp_update(b, torch, inputs, runtime, dev, peaks, hp)
    elif args.only == "decode":
        out = decode_bandwidth(b, torch, inputs, dev, peaks, n_blocks=args.decode_blocks)
    elif args.only == "config2":
        out = config_stack32(b, torch, inputs, runtime, dev, peaks, hp)
    else:
        out = config_70b(b, torch, inputs, runtime, dev, peaks, hp)
    print(json.dumps({args.only: out}))
    return 0


def cublas_same_shapes(torch, blocks, projections, T, steps):
    """TFLOP/s of torch.matmul (cuBLAS) on the frozen-weight products of the timed blocks: x W0^T and dY W0
    for every projection, rotating over the same blocks, CUDA events around `steps` passes."""
    def one_pass(blk):
        for x, dY, W0 in zip(blk.x, blk.dY, blk.W0):
            torch.matmul(x, W0.t())
            torch.matmul(dY, W0)
    for blk in blocks[:2]:
        one_pass(blk)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        one_pass(blocks[i % len(blocks)])
    e1.record()
    torch.cuda.synchronize()
    flops = sum(4 * T * di * do for _, di, do in projections) * steps
    return flops / (e0.elapsed_time(e1) * 1e-3) / 1e12


def timed_updates(b, torch, runtime, arg_list, ws, batch, epochs, hp, steps, warmup):
    """warmup + steps chunk updates rotating over arg_list, CUDA events around the timed ones, library events
    around the fused GEMM kernel's launches, clocks sampled meanwhile."""
    taken = [0] * len(arg_list)

    def step(i):
        k = i % len(arg_list)
        taken[k] = b.templora_update_block_batched(arg_list[k], batch, epochs, hp["lr"], hp["beta1"], hp["beta2"],
                                                   hp["eps"], hp["weight_decay"], taken[k], ws)
    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    for k in range(b.N_KINDS):
        b.templora_timing_read(k, reset=True)
    b.templora_timing_enable([b.KIND_TC_MAIN])
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with runtime.ClockSampler(torch.cuda.current_device()) as clk:
        e0.record(stream)
        for i in range(steps):
            step(i)
        e1.record(stream)
        torch.cuda.synchronize()
    b.templora_timing_enable(False)
    ms_main, n_main, _ = b.templora_timing_read(b.KIND_TC_MAIN, reset=True)
    code, where = b.templora_read_device_status(ws)
    assert code == 0, f"device status {code} at {where}"
    return e0.elapsed_time(e1) / 1e3, clk.summary(), ms_main, n_main


def config_stack32(b, torch, inputs, runtime, dev, peaks, hp, n_blocks=32, epochs=2, steps=6, warmup=3):
    """The full chunk update over 32 stacked 7B-shaped blocks (distinct frozen weights and LoRA state per block,
    x / dY / y / dX per projection type shared by the blocks), 2 epochs, in ONE templora_update_block call."""
    c = inputs.CONFIGS[2]
    T, r, s, projections = c["T"], c["r"], c["s"], c["projections"]
    shared, stack = None, []
    for i in range(n_blocks):
        blk = runtime.Block(b, 0, f"cfg2/stack{i}", projections, T, r, s, "bf16", dev, shared_io=shared)
        shared = shared or blk.io
        stack.append(blk)
    cat = lambda f: [t for blk in stack for t in f(blk)]
    lins = cat(lambda k: k.lins)
    call = b.UpdateBlockArgs(lins, cat(lambda k: k.A_desc), cat(lambda k: k.B_desc), cat(lambda k: k.x),
                             cat(lambda k: k.dY), cat(lambda k: k.y), cat(lambda k: k.dX))
    ws = b.alloc_workspace(b.templora_update_block_workspace_bytes(lins, T), dev)
    seconds, clocks, ms_main, n_main = timed_updates(b, torch, runtime, [call], ws, T, epochs, hp, steps, warmup)
    regime = pick_regime(seconds, clocks)
    flops_update = block_flops(projections, T, r) * epochs * n_blocks
    tf_update = flops_update * steps / seconds / 1e12
    tf_main = main_kernel_flops(projections, T, r) * epochs * n_blocks * steps / (ms_main * 1e-3) / 1e12 if n_main else None
    return {"workload": f"{n_blocks} stacked llama2_7b blocks x 7 LoRA projections, T={T}, r={r}, s={s}, {epochs} epochs, one templora_update_block call per chunk update",
            "updates_timed": steps, "warmup": warmup, "ms_per_chunk_update": 1e3 * seconds / steps,
            "chunk_tokens_per_s": T * steps / seconds, "token_epochs_per_s": T * epochs * steps / seconds,
            "tflops": tf_update, "regime": regime, **fractions(tf_update, peaks, regime),
            "pair_kernel_tflops": tf_main,
            "pair_kernel": {k: v for k, v in fractions(tf_main, peaks, regime).items()},
            "target_chunk_tokens_per_s_at_0.6_of_nominal": T / (flops_update / (0.6 * NOMINAL_TFLOPS * 1e12)),
            "clocks": clocks}


def config_70b(b, torch, inputs, runtime, dev, peaks, hp, steps=12, warmup=3):
    """One Llama-2-70B-shaped block (GQA: k, v project to 1024), T = 4096, one epoch per step."""
    c = inputs.CONFIGS[4]
    T, r, s, projections = c["T"], c["r"], c["s"], c["projections"]
    blk = runtime.Block(b, 0, "cfg4/blk", projections, T, r, s, "bf16", dev)
    ws = b.alloc_workspace(b.templora_update_block_workspace_bytes(blk.lins, T), dev)
    seconds, clocks, ms_main, n_main = timed_updates(b, torch, runtime, [blk.args], ws, T, 1, hp, steps, warmup)
    regime = pick_regime(seconds, clocks)
    tf_step = block_flops(projections, T, r) * steps / seconds / 1e12
    tf_main = main_kernel_flops(projections, T, r) * steps / (ms_main * 1e-3) / 1e12 if n_main else None
    return {"workload": f"llama2_70b block: 7 LoRA projections (q,o 8192x8192; k,v 8192->1024; gate,up 8192->28672; down 28672->8192), T={T}, r={r}, s={s}, fwd+bwd+AdamW",
            "steps": steps, "warmup": warmup, "ms_per_step": 1e3 * seconds / steps, "tokens_per_s": T * steps / seconds,
            "tflops": tf_step, "regime": regime, **fractions(tf_step, peaks, regime),
            "pair_kernel_tflops": tf_main, "pair_kernel": {k: v for k, v in fractions(tf_main, peaks, regime).items()},
            "l2": "one block: its frozen weights (1.7 GB) and activations (2.7 GB) exceed the 126 MB L2",
            "clocks": clocks}


def parallel_deployment(b, torch, runtime, blk, hp, update_sms=116, decode_sms=32, n_updates=20):
    """The paper's parallelized deployment on one GPU: chunk updates (7B block, T=1024) back to back on
    one stream while single-token decode steps of the same block run on another, with the SMs split
    between the two sides: fixed disjoint groups of SMs (templora_sm_partition_create) and, for comparison,
    per-stream caps on the grid sizes alone.  Reports both rates alone and side by side."""
    out = _parallel_deployment(b, torch, runtime, blk, hp, update_sms, decode_sms, n_updates, True)
    if out["sm_partition"]:
        caps = _parallel_deployment(b, torch, runtime, blk, hp, update_sms, decode_sms, n_updates, False)
        out["caps_only"] = {k: caps[k] for k in ("update_ms_alone_capped", "decode_step_us_alone_capped",
                                                 "update_ms_side_by_side", "decode_step_us_side_by_side")}
    return out


def _parallel_deployment(b, torch, runtime, blk, hp, update_sms, decode_sms, n_updates, partition):
    dep = runtime.ParallelDeployment(b, blk, n_tokens=1, update_sms=update_sms, decode_sms=decode_sms,
                                     partition=partition)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    try:
        def timed(fn, stream, reps):
            fn(); stream.synchronize()
            e0, e1 = ev(), ev()
            e0.record(stream)
            for _ in range(reps):
                fn()
            e1.record(stream)
            stream.synchronize()
            return e0.elapsed_time(e1) / reps
        upd = lambda: dep.start_update(1, hp)
        upd_alone_ms = timed(upd, dep.update_stream, n_updates)
        dec_alone_ms = timed(dep.decode_step, dep.decode_stream, 50)
        # side by side: enqueue the updates, then decode steps (each with its own event) well past their end;
        # only the decode steps that finished while the updates were still running count as contended
        torch.cuda.synchronize()
        e0, e1 = ev(), ev()
        n_dec = int(2.5 * n_updates * upd_alone_ms / max(dec_alone_ms, 1e-6)) + 8
        marks = [ev() for _ in range(n_dec + 1)]
        e0.record(dep.update_stream)
        for _ in range(n_updates):
            upd()
        e1.record(dep.update_stream)
        marks[0].record(dep.decode_stream)
        for i in range(n_dec):
            dep.decode_step()
            marks[i + 1].record(dep.decode_stream)
        torch.cuda.synchronize()
        upd_end = marks[0].elapsed_time(e1)                      # update end on the decode stream's clock
        ends = [marks[0].elapsed_time(m) for m in marks[1:]]
        contended = [i for i, t in enumerate(ends) if t <= upd_end]
        dec_side_us = (ends[contended[-1]] / (contended[-1] + 1) * 1e3) if contended else None
        dep.publish()
        torch.cuda.synchronize()
        return {"update_sms": dep.update_sms, "decode_sms": dep.decode_sms, "sm_partition": dep.partition is not None,
                "update_ms_alone_capped": upd_alone_ms, "decode_step_us_alone_capped": dec_alone_ms * 1e3,
                "update_ms_side_by_side": e0.elapsed_time(e1) / n_updates,
                "decode_step_us_side_by_side": dec_side_us, "decode_steps_during_updates": len(contended),
                "what": "7B block: chunk updates (T=1024) back to back on one stream, single-token decode steps of the "
                        "same block on another; 'alone' figures keep the SM split; caps_only: ordinary streams with "
                        "per-stream caps on the persistent kernels' grids instead of disjoint SM groups"}
    finally:
        dep.close()


def mlp_update(b, torch, inputs, runtime, dev, peaks, hp, T=1024, r=64, steps=40, warmup=5, n_rot=3):
    """templora_update_mlp on the 7B block's MLP (gate, up 4096 -> 11008, down 11008 -> 4096; T = 1024): gate and up as
    one GEMM whose epilogue writes gate, up and h = SiLU(gate) * up, dgate and dup written by the epilogue of the down
    projection's input gradient.  Beside it: what the stand-alone gating kernels take at the same shape (the two
    [T, d_ff] round trips the fused call does not make) and how many of them the timed calls launched (none)."""
    d, d_ff, s = 4096, 11008, 2.0
    projs = [("gate", d, d_ff), ("up", d, d_ff), ("down", d_ff, d)]
    sets = []
    for i in range(n_rot):
        blk = runtime.Block(b, 0, f"mlp{i}", projs, T, r, s, "bf16", dev, with_dX=False)
        bufs = dict(x=blk.x[0], dY=blk.dY[2], y=blk.y[2],
                    gate=torch.empty((T, d_ff), dtype=torch.bfloat16, device=dev),
                    up=torch.empty((T, d_ff), dtype=torch.bfloat16, device=dev),
                    h=torch.empty((T, d_ff), dtype=torch.bfloat16, device=dev),
                    dX=torch.empty((T, d), dtype=torch.bfloat16, device=dev))
        sets.append((blk, bufs))
    ws = b.alloc_workspace(b.templora_update_mlp_workspace_bytes(sets[0][0].lins, T), dev)
    step = [0] * n_rot

    def one(i):
        blk, q = sets[i % n_rot]
        step[i % n_rot] = b.templora_update_mlp(blk.lins, blk.A_desc, blk.B_desc, q["x"], q["dY"], q["gate"], q["up"], q["h"],
                                                q["y"], q["dX"], 1, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
                                                hp["weight_decay"], step[i % n_rot], ws)
    for i in range(warmup):
        one(i)
    torch.cuda.synchronize()
    b.templora_timing_enable(False)
    for k in range(b.N_KINDS):
        b.templora_timing_read(k, reset=True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with runtime.ClockSampler(torch.cuda.current_device()) as clk:
        e0.record()
        for i in range(steps):
            one(i)
        e1.record()
        torch.cuda.synchronize()
    clocks = clk.summary()
    assert b.templora_read_device_status(ws)[0] == 0
    launches = {k: b.templora_timing_read(k)[2] for k in range(b.N_KINDS)}
    sec = e0.elapsed_time(e1) / 1e3 / steps
    flops = block_flops(projs, T, r)
    # the stand-alone gating kernels at this shape, for scale
    g = sets[0][1]
    scratch = [torch.empty((T, d_ff), dtype=torch.bfloat16, device=dev) for _ in range(2)]
    def timed(fn, reps=20):
        fn(); torch.cuda.synchronize()
        a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        c.record(); torch.cuda.synchronize()
        return a.elapsed_time(c) / reps * 1e3
    fwd_us = timed(lambda: b.templora_swiglu_fwd(g["gate"], g["up"], scratch[0]))
    bwd_us = timed(lambda: b.templora_swiglu_bwd(g["gate"], g["up"], g["h"], scratch[0], scratch[1]))
    regime = pick_regime(sec * steps, clocks)
    return {"workload": f"MLP of a llama2_7b block (gate, up {d}->{d_ff}, down {d_ff}->{d}), T={T}, r={r}, one "
                        "templora_update_mlp call per step (forward, backward, AdamW on the six LoRA matrices)",
            "steps": steps, "ms_per_step": sec * 1e3, "tokens_per_s": T / sec, "tflops": flops / sec / 1e12,
            **fractions(flops / sec / 1e12, peaks, regime), "regime": regime,
            "gating_kernel_launches_in_timed_calls": int(launches[b.KIND_BLOCK_OPS]),
            "standalone_gating_us_at_this_shape": {"swiglu_fwd": fwd_us, "swiglu_bwd": bwd_us},
            "launches_per_step": sum(launches.values()) / steps, "clocks": clocks}


def block_ops_bandwidth(b, torch, inputs, dev, peaks, T=4096, reps=20):
    """HBM throughput of the SiLU-gating and RMSNorm kernels at 7B widths (bf16; T rows of 11008 for the
    gating, 4 T rows of 4096 for the norm so that a launch outlasts the host's call overhead; four buffer
    sets in rotation so that each launch's tensors come from DRAM).  Bytes = every tensor read or written once."""
    Tn = 4 * T
    n_rot = 4
    mk = lambda tag, shape: inputs.make_tensor(0, "blockops", tag, shape, "normal", 1.0, "bf16", dev)
    sets = [dict(g=mk(f"g{i}", (T, 11008)), u=mk(f"u{i}", (T, 11008)), dh=mk(f"dh{i}", (T, 11008)),
                 o0=torch.empty((T, 11008), dtype=torch.bfloat16, device=dev),
                 o1=torch.empty((T, 11008), dtype=torch.bfloat16, device=dev),
                 x=mk(f"x{i}", (Tn, 4096)), dy=mk(f"dy{i}", (Tn, 4096)),
                 y=torch.empty((Tn, 4096), dtype=torch.bfloat16, device=dev)) for i in range(n_rot)]
    w = inputs.make_tensor(0, "blockops", "w", (4096,), "uniform", 1.0, "bf16", dev)
    ops = {
        "swiglu_fwd": (lambda s: b.templora_swiglu_fwd(s["g"], s["u"], s["o0"]), 3 * T * 11008 * 2),
        "swiglu_bwd": (lambda s: b.templora_swiglu_bwd(s["g"], s["u"], s["dh"], s["o0"], s["o1"]), 5 * T * 11008 * 2),
        "rmsnorm_fwd": (lambda s: b.templora_rmsnorm_fwd(s["x"], w, 1e-5, s["y"]), 2 * Tn * 4096 * 2),
        "rmsnorm_bwd": (lambda s: b.templora_rmsnorm_bwd(s["x"], w, s["dy"], 1e-5, s["y"]), 3 * Tn * 4096 * 2),
    }
    out = {"rows_gating": T, "rows_norm": Tn, "dtype": "bf16"}
    for name, (fn, nbytes) in ops.items():
        for s in sets:
            fn(s)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            for s in sets:
                fn(s)
        e1.record()
        torch.cuda.synchronize()
        sec = e0.elapsed_time(e1) / 1e3 / (reps * n_rot)
        out[name] = {"us": sec * 1e6, "GBps": nbytes / sec / 1e9, "frac_of_measured_hbm": nbytes / sec / 1e9 / peaks["hbm"]}
    return out


def decode_bandwidth(b, torch, inputs, dev, peaks, n_blocks=32, reps=5):
    """Decode-time forward of a 7B-shaped block for 1, 4 and 16 tokens, rotating over 32 blocks with
    distinct weights so that no W0 byte is served from L2.  GB/s = streamed W0, A, B bytes / time."""
    c = inputs.CONFIGS[3]
    r, s, projections = c["r"], c["s"], c["projections"]
    blocks = []
    for i in range(n_blocks):
        lins = []
        for name, d_in, d_out in projections:
            t = f"dec{i}/{name}"
            W0 = inputs.make_tensor(0, t, "W0", (d_out, d_in), "normal", d_in ** -0.5, "bf16", dev)
            A = inputs.make_tensor(0, t, "A", (r, d_in), "uniform", d_in ** -0.5, "bf16", dev)
            B = inputs.make_tensor(0, t, "B", (d_out, r), "normal", 0.02, "bf16", dev)
            lins.append(b.linear_desc(W0, A, B, s))
        blocks.append(lins)
    bytes_per_block = sum(inputs.decode_bytes(di, do, r) for _, di, do in projections)
    ws_bytes = max([b.templora_workspace_bytes(l, 16) for l in blocks[0]] +
                   [b.templora_decode_block_workspace_bytes(blocks[0][i:j]) for i, j in ((0, 7), (0, 3), (3, 4), (4, 6), (6, 7))])
    ws = b.alloc_workspace(ws_bytes, dev)
    out = {}
    for n in c["decode_tokens"]:
        xs = {di: inputs.make_tensor(0, "dec", f"x{n}-{di}", (n, di), "normal", 1.0, "bf16", dev) for di in (4096, 11008)}
        ys = {do: torch.empty((n, do), dtype=torch.bfloat16, device=dev) for do in (4096, 11008)}

        def sweep_single():
            for lins in blocks:
                for lin in lins:
                    b.templora_decode_fwd(lin, xs[lin.d_in], ys[lin.d_out], ws)

        def sweep_block():
            for a in block_args:
                b.templora_decode_block_fwd(a, ws)

        block_args = [b.DecodeBlockArgs(lins, [xs[l.d_in] for l in lins], [ys[l.d_out] for l in lins]) for lins in blocks]
        # the order a real decoder block imposes: q,k,v share their input; o, then gate and up, then down
        # each wait for the step before: four grouped calls per block
        group_args = [[b.DecodeBlockArgs(lins[i:j], [xs[l.d_in] for l in lins[i:j]], [ys[l.d_out] for l in lins[i:j]])
                       for i, j in ((0, 3), (3, 4), (4, 6), (6, 7))] for lins in blocks]

        def sweep_groups():
            for ga in group_args:
                for a in ga:
                    b.templora_decode_block_fwd(a, ws)

        res = {}
        for label, sweep, calls_per_block in (("per_projection_calls", sweep_single, 7),
                                              ("four_dependent_group_calls", sweep_groups, 4),
                                              ("one_call_per_block", sweep_block, 1)):
            sweep()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                sweep()
            e1.record()
            torch.cuda.synchronize()
            sec = e0.elapsed_time(e1) / 1e3 / (reps * n_blocks)
            gbs = bytes_per_block / sec / 1e9
            res[label] = {"us_per_block": sec * 1e6, "GBps": gbs, "frac_of_measured_hbm": gbs / peaks["hbm"],
                          "frac_of_nominal_8000": gbs / 8000.0, "calls_per_block": calls_per_block}
            # where that time goes.  Host: wall clock around one sweep of calls that nothing waits for (the
            # GPU is idle at its start, so the launch queue never fills: pure marshalling + launch cost).
            # Device: the library's own events around each kernel launch, summed per block (this run loses
            # the overlap of one launch's set-up with its predecessor's tail, so it is an upper bound on
            # the kernels' share of the back-to-back figure above).
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            sweep()
            host = time.perf_counter() - t0
            torch.cuda.synchronize()
            for k in (b.KIND_TC_DECODE, b.KIND_DECODE_FINISH):
                b.templora_timing_read(k, reset=True)
            b.templora_timing_enable([b.KIND_TC_DECODE, b.KIND_DECODE_FINISH])
            sweep()
            torch.cuda.synchronize()
            b.templora_timing_enable(False)
            ms_tc, n_tc, _ = b.templora_timing_read(b.KIND_TC_DECODE, reset=True)
            ms_fin, n_fin, _ = b.templora_timing_read(b.KIND_DECODE_FINISH, reset=True)
            res[label]["host_us_per_call"] = host * 1e6 / (n_blocks * calls_per_block)
            res[label]["host_us_per_block"] = host * 1e6 / n_blocks
            res[label]["device_kernel_us_per_block"] = 1e3 * (ms_tc + ms_fin) / n_blocks
            res[label]["device_kernel_GBps"] = bytes_per_block / ((ms_tc + ms_fin) * 1e-3 / n_blocks) / 1e9
            res[label]["kernel_launches_per_block"] = (n_tc + n_fin) / n_blocks
        out[f"n{n}"] = res
    # the order a decoder block imposes (q,k,v -> o -> gate,up -> down) is the figure a serving loop can realise;
    # one call per block treats the seven projections as independent and is the kernel's own ceiling
    out["headline"] = {"mode": "four_dependent_group_calls",
                       **{f"n{n}": {k: out[f"n{n}"]["four_dependent_group_calls"][k]
                                    for k in ("us_per_block", "GBps", "frac_of_measured_hbm", "frac_of_nominal_8000")}
                          for n in c["decode_tokens"]}}
    code, where = b.templora_read_device_status(ws)
    assert code == 0, f"decode device status {code} at {where}"
    out["bytes_per_block"] = bytes_per_block
    out["hbm_peak_GBps"] = peaks["hbm"]
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="timed steps (default 200; 20 for --impl reference)")
    ap.add_argument("--warmup", type=int, default=None, help="untimed steps before them (default 10; 3 for --impl reference)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--blocks", type=int, default=N_ROTATE, help="distinct blocks the steps rotate over")
    ap.add_argument("--model", default="llama2_7b", choices=["llama2_7b", "llama2_13b", "llama2_70b", "mistral_7b", "yi_6b"],
                    help="block shape (default: the metric's workload)")
    ap.add_argument("--chunk", type=int, default=1024, help="tokens in the chunk (paper: 1024, 2048, 4096)")
    ap.add_argument("--batch", type=int, default=0, help="tokens per optimizer step (default: the whole chunk)")
    ap.add_argument("--rank", type=int, default=64)
    ap.add_argument("--epochs", type=int, default=1)
    ap.add_argument("--stacked-blocks", type=int, default=0,
                    help="update this many blocks in one call (32 with --epochs 2: the full 7B-stack chunk update)")
    ap.add_argument("--dropout", type=float, default=0.0, help="LoRA dropout probability (paper: 0.05; the metric's workload: 0)")
    ap.add_argument("--shared-input", action="store_true",
                    help="q,k,v and gate,up read one input each and get one summed dX each (templora_linear_t.input_group)")
    ap.add_argument("--no-decode", action="store_true")
    ap.add_argument("--decode-blocks", type=int, default=32, help="distinct blocks the decode measurement rotates over")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-parallel", action="store_true", help="skip the parallelized-deployment measurement")
    ap.add_argument("--no-configs", action="store_true", help="skip the 32-block stack and the 70B block")
    ap.add_argument("--only", default=None, choices=["block_ops", "decode", "config2", "config4", "mlp"],
                    help="run one side measurement alone and print its JSON object (profiling aid; not the bench line)")
    args = ap.parse_args()
    reference = args.impl == "reference"
    if args.steps is None:
        args.steps = 20 if reference else 200
    if args.warmup is None:
        args.warmup = 3 if reference else 10
    if reference:
        return run_reference(args)
    if args.only:
        return run_only(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started plainly: be the launcher, one worker per GPU (what torch.distributed.run would start)
        from paper_2401_11504_b200 import runtime
        return runtime.spawn_replicas([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], args.gpus)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
