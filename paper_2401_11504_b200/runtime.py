"""Host-side plumbing around the library: building a block of LoRA-augmented projections on a
device, rank bookkeeping for replicated runs, and clock sampling.  No arithmetic of the method.

Multi-GPU: the path does not shard (one GPU holds a whole block and its chunk); N GPUs run N
independent replicas.  The only cross-rank steps are a barrier around the timed region and a max
over ranks of the measured time, both through torch.distributed (nccl on GPUs, gloo on CPU).
"""
import os
import socket
import subprocess
import threading
import time

import torch
import torch.distributed as dist

from . import inputs


# ------------------------------------------------------------------ ranks
class Ranks:
    """World bookkeeping for replicated runs; a single process is world_size 1 without a group."""

    def __init__(self, backend=None):
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.group = False
        if self.world > 1:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29531")
            backend = backend or ("nccl" if torch.cuda.is_available() else "gloo")
            if backend == "nccl":
                torch.cuda.set_device(self.local_rank)
            dist.init_process_group(backend=backend, rank=self.rank, world_size=self.world)
            self.group = True
            self.backend = backend

    def _dev(self):
        return torch.device("cuda", self.local_rank) if self.group and self.backend == "nccl" else torch.device("cpu")

    def barrier(self):
        if self.group:
            dist.barrier()

    def max_over_ranks(self, value):
        if not self.group:
            return float(value)
        t = torch.tensor([float(value)], dtype=torch.float64, device=self._dev())
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def sum_over_ranks(self, value):
        if not self.group:
            return float(value)
        t = torch.tensor([float(value)], dtype=torch.float64, device=self._dev())
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return float(t.item())

    def close(self):
        if self.group:
            dist.destroy_process_group()
            self.group = False


def aggregate_throughput(units_per_rank, seconds_this_rank, ranks):
    """Whole-job throughput of replicated work: units of all ranks / slowest rank's time."""
    total_units = ranks.sum_over_ranks(units_per_rank)
    slowest = ranks.max_over_ranks(seconds_this_rank)
    return total_units / slowest, slowest


def _free_port():
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def spawn_replicas(argv, n, timeout_s=3600):
    """Start n copies of the command argv as the ranks of one job on this node, one per GPU: RANK and
    LOCAL_RANK 0..n-1, WORLD_SIZE n, rendezvous on 127.0.0.1 at a free port (what torch.distributed.run
    would set).  Rank 0's standard output is passed through (it prints the job's one result line); the
    other ranks' output is dropped, everybody's standard error is passed through.  Returns the first
    non-zero exit code, or 0.  A rank that fails ends the others: they would wait in the rendezvous for ever."""
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()), WORLD_SIZE=str(n))
    procs = []
    for rank in range(n):
        e = dict(env, RANK=str(rank), LOCAL_RANK=str(rank))
        procs.append(subprocess.Popen(list(argv), env=e, stdout=None if rank == 0 else subprocess.DEVNULL))
    deadline = time.time() + timeout_s
    rc = 0
    pending = list(procs)
    while pending:
        for p in list(pending):
            code = p.poll()
            if code is None:
                continue
            pending.remove(p)
            if code != 0 and rc == 0:
                rc = code
        if rc != 0 or time.time() > deadline:
            for p in pending:
                p.terminate()
            for p in pending:
                try:
                    p.wait(timeout=10)
                except subprocess.TimeoutExpired:
                    p.kill()
            if rc == 0:
                rc = 124
            break
        time.sleep(0.05)
    return rc


# ------------------------------------------------------------------ block construction
class Block:
    """One block of LoRA-augmented projections resident on a device, with optimizer state."""

    def __init__(self, b, seed, tag, projections, T, r, s, dtype="bf16", device="cuda", with_dX=True,
                 shared_io=None, dropout_p=0.0, input_groups=None):
        """input_groups: lists of projection names that read the same input (e.g. [["q", "k", "v"],
        ["gate", "up"]]): the members share the first member's x and dX tensors, and dX receives the sum
        of their input gradients (templora_linear_t.input_group)."""
        group_of = {}
        for gi, names in enumerate(input_groups or []):
            for nm in names:
                group_of[nm] = (gi + 1, names[0])
        self.T, self.r, self.s, self.dtype = T, r, s, dtype
        self.names = [p[0] for p in projections]
        self.W0, self.state, self.lins, self.A_desc, self.B_desc = [], [], [], [], []
        self.x, self.dY, self.y, self.dX = [], [], [], []
        self.io = {}
        td = torch.bfloat16 if dtype == "bf16" else torch.float32
        for name, d_in, d_out in projections:
            t = f"{tag}/{name}"
            W0 = inputs.make_tensor(seed, t, "W0", (d_out, d_in), "normal", d_in ** -0.5, dtype, device)
            st = {}
            for nm, shape, kind, scale in (("A", (r, d_in), "uniform", d_in ** -0.5), ("B", (d_out, r), "normal", 0.02)):
                w = inputs.make_tensor(seed, t, nm, shape, kind, scale, dtype, device)
                master = w.float().contiguous()
                st[nm] = dict(master=master, m=torch.zeros_like(master), v=torch.zeros_like(master),
                              grad=torch.zeros_like(master), work=w.contiguous() if dtype == "bf16" else None)
            a = st["A"]["work"] if dtype == "bf16" else st["A"]["master"]
            bb = st["B"]["work"] if dtype == "bf16" else st["B"]["master"]
            self.W0.append(W0)
            self.state.append(st)
            self.lins.append(b.linear_desc(W0, a, bb, s, dropout_p=dropout_p,
                                           dropout_seed=inputs._key(seed, t, "dropout") & ((1 << 64) - 1),
                                           input_group=group_of.get(name, (0, None))[0]))
            self.A_desc.append(b.param_desc(st["A"]["master"], st["A"]["m"], st["A"]["v"], st["A"]["grad"], st["A"]["work"]))
            self.B_desc.append(b.param_desc(st["B"]["master"], st["B"]["m"], st["B"]["v"], st["B"]["grad"], st["B"]["work"]))
            if shared_io is not None:
                io = shared_io[name]
            else:
                io = dict(x=inputs.make_tensor(seed, t, "x", (T, d_in), "normal", 1.0, dtype, device),
                          dY=inputs.make_tensor(seed, t, "dY", (T, d_out), "normal", 1.0, dtype, device))
                io["y"] = torch.empty((T, d_out), dtype=td, device=device)
                io["dX"] = torch.empty((T, d_in), dtype=td, device=device) if with_dX else None
                if name in group_of and group_of[name][1] != name:   # reads (and differentiates into) the leader's
                    io["x"], io["dX"] = self.io[group_of[name][1]]["x"], self.io[group_of[name][1]]["dX"]
            self.io[name] = io
            self.x.append(io["x"]); self.dY.append(io["dY"]); self.y.append(io["y"]); self.dX.append(io["dX"])
        self.args = b.UpdateBlockArgs(self.lins, self.A_desc, self.B_desc, self.x, self.dY, self.y,
                                      self.dX if with_dX else None)

    def n_lora_params(self):
        return sum(st["A"]["master"].numel() + st["B"]["master"].numel() for st in self.state)


# ------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while a region runs."""

    def __init__(self, cuda_index=0, period_s=0.005):
        self.index, self.period = cuda_index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            try:  # NVML numbers GPUs by PCI order, CUDA by visibility: match on the PCI address
                pr = torch.cuda.get_device_properties(cuda_index)
                bus_id = f"{pr.pci_domain_id:08X}:{pr.pci_bus_id:02X}:{pr.pci_device_id:02X}.0"
                self._h = pynvml.nvmlDeviceGetHandleByPciBusId(bus_id.encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(cuda_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None

    _REASONS = (("hw_slowdown", 0x8), ("sw_power_cap", 0x4), ("hw_thermal_slowdown", 0x40),
                ("sw_thermal_slowdown", 0x20), ("hw_power_brake", 0x80), ("sync_boost", 0x10))

    def _once(self):
        nv = self._nv
        self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
        try:
            mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
        except Exception:
            mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
        for name, bit in self._REASONS:
            if mask & bit:
                self.reasons.add(name)

    def _run(self):
        while not self._stop.is_set():
            try:
                self._once()
            except Exception:
                break
            time.sleep(self.period)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2.0)
            try:
                self._once()
            except Exception:
                pass

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["clock sampling unavailable"]}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


# ------------------------------------------------------------------ parallelized deployment
class ParallelDeployment:
    """Chunk update and decode side by side on one GPU (the paper's parallelized deployment:
    the module is updated elsewhere while generation goes on, then swapped in).

    The update runs on its own stream and trains the block's working copies of A and B; decode runs
    on another stream and reads separate *serving* copies, so it always sees a complete module.
    publish() swaps the new module in at a decode-step boundary: on the decode stream, after the
    update's completion event, the working copies are copied over the serving copies (10 MB for a
    7B-shaped block).  The two streams run on disjoint groups of SMs (templora_sm_partition_create:
    decode_sms for the decode stream, the rest for the update); with partition=False, or where the
    driver offers no SM partitioning, they are ordinary streams with per-stream SM caps.
    Orchestration only: every product runs in the library's kernels.
    """

    def __init__(self, b, blk, n_tokens=1, update_sms=116, decode_sms=32, device="cuda", partition=True):
        self.b, self.blk, self.n = b, blk, n_tokens
        self.partition = None
        if partition:
            try:
                self.partition = b.templora_sm_partition_create(decode_sms)
            except b.TemploraError as e:
                if e.code != b.ERR_UNSUPPORTED:
                    raise
        if self.partition is not None:
            self.decode_stream = torch.cuda.ExternalStream(self.partition.stream_first, device=device)
            self.update_stream = torch.cuda.ExternalStream(self.partition.stream_rest, device=device)
            self.decode_sms, self.update_sms = self.partition.sms_first, self.partition.sms_rest
        else:
            self.update_stream = torch.cuda.Stream(device=device)
            self.decode_stream = torch.cuda.Stream(device=device)
            b.templora_set_stream_sm_limit(self.update_stream, update_sms)
            b.templora_set_stream_sm_limit(self.decode_stream, decode_sms)
            self.decode_sms, self.update_sms = decode_sms, update_sms
        self.serving = [(st["A"]["work"].clone(), st["B"]["work"].clone()) for st in blk.state]
        self.lins = [b.linear_desc(W0, a, bb, blk.s) for W0, (a, bb) in zip(blk.W0, self.serving)]
        td = blk.x[0].dtype
        dt = "bf16" if td == torch.bfloat16 else "f32"
        self.x = [inputs.make_tensor(0, "deploy", f"x{i}", (n_tokens, l.d_in), "normal", 1.0, dt, device)
                  for i, l in enumerate(self.lins)]
        self.y = [torch.empty((n_tokens, l.d_out), dtype=td, device=device) for l in self.lins]
        self.dec_args = b.DecodeBlockArgs(self.lins, self.x, self.y)
        self.ws_dec = b.alloc_workspace(b.templora_decode_block_workspace_bytes(self.lins), device)
        self.ws_upd = b.alloc_workspace(b.templora_update_block_workspace_bytes(blk.lins, blk.T), device)
        self.update_done = torch.cuda.Event()
        self.published = torch.cuda.Event()
        self.published.record(self.decode_stream)
        self.step = 0

    def start_update(self, epochs, hp, batch=None):
        """Enqueue the chunk update on the update stream (returns at once)."""
        self.update_stream.wait_event(self.published)   # the last publish has read the working copies
        self.step = self.b.templora_update_block_batched(
            self.blk.args, batch or self.blk.T, epochs, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
            hp["weight_decay"], self.step, self.ws_upd, stream=self.update_stream)
        self.update_done.record(self.update_stream)

    def decode_step(self):
        """One decode-time forward of the whole block with the serving module."""
        self.b.templora_decode_block_fwd(self.dec_args, self.ws_dec, stream=self.decode_stream)

    def publish(self):
        """Swap the updated module in between two decode steps."""
        self.decode_stream.wait_event(self.update_done)
        with torch.cuda.stream(self.decode_stream):
            for st, (sa, sb) in zip(self.blk.state, self.serving):
                sa.copy_(st["A"]["work"], non_blocking=True)
                sb.copy_(st["B"]["work"], non_blocking=True)
        self.published.record(self.decode_stream)

    def close(self):
        if self.partition is not None:
            self.b.templora_sm_partition_destroy(self.partition)   # synchronises and destroys both streams
            self.partition = None
            return
        self.b.templora_set_stream_sm_limit(self.update_stream, 0)
        self.b.templora_set_stream_sm_limit(self.decode_stream, 0)
