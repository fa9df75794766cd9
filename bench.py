#!/usr/bin/env python
"""Benchmark of the Few-Bit Backward hot path on B200.

One "step" is one pass of the whole hot path over one batch of the headline
workload: for every bit width of the workload, the fused forward kernel
(activation + bucketize + pack) followed by the backward kernel (unpack +
level lookup + multiply).  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c3|c2|c4|c1]
                    [--scaling weak|strong]

N > 1: one rank per GPU.  Under torchrun (WORLD_SIZE set) the script is a rank; started plainly with
--gpus N > 1 it re-launches itself under torch.distributed.run with N ranks on 127.0.0.1.  The path is
elementwise, so the ranks share nothing but the barrier and the max-reduction of the time: with
--scaling weak (default) every rank processes its own tensor of the workload's shape, with --scaling
strong ONE tensor of the workload is cut with workloads.shard_range on multiples of 32 elements and
every rank runs its shard; `checksum` (a sum over the bit patterns of every output) is then the same
for every N.
"""
from __future__ import annotations

import argparse
import dataclasses
import datetime
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2202_00441_b200 import workloads as wl  # noqa: E402

METRIC = "fused fwd+pack / unpack+bwd elements/s and HBM GB/s vs ~8 TB/s peak"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


# ----------------------------------------------------------------------------
# helpers
# ----------------------------------------------------------------------------
def elem_size(case: wl.Case) -> int:
    return 4 if case.dtype == "f32" else 2


def algorithmic_bytes(case: wl.Case, n: int, bits: int) -> float:
    """Per kernel launch (forward: x in, y out, codes out; backward: codes in,
    grad_out in, grad_in out): n * (2 * sizeof(T) + bits / 8)."""
    return n * (2 * elem_size(case) + bits / 8.0)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""

    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.index)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        """Summary of the samples; with wall-clock bounds, of those taken between them (the timed region)."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = []
        try:
            rows = open(self.path).read().splitlines()
            os.unlink(self.path)
        except Exception:
            pass
        out = self._summarise(rows, t_begin, t_end, out, "timed region")
        if out["samples"] == 0 and t_begin is not None:      # region shorter than the sampling period
            out = self._summarise(rows, t_begin - 0.25, t_end + 0.25, out, "within 0.25 s of the timed region")
        return out

    @staticmethod
    def _summarise(rows, t_begin, t_end, out, window):
        clocks, reasons, mx = [], set(), None
        try:
            for line in rows:
                f = [c.strip() for c in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    if t_begin is not None:
                        ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                        if not (t_begin <= ts <= t_end):
                            continue
                    clocks.append(float(f[1])); mx = float(f[2])
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
        except Exception:
            pass
        if clocks:
            out = dict(out, sm_mhz=statistics.median(clocks), sm_max_mhz=mx, reasons=sorted(reasons), samples=len(clocks),
                       window=window)
        return out


def dist_setup(n_gpus: int):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        # the communicator log shows the rank count; it goes to a file per process, never to stdout
        # (stdout carries the one JSON line)
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        os.environ.setdefault("NCCL_DEBUG_FILE", os.path.join(tempfile.gettempdir(), "fewbit_bench_nccl_%h_%p.log"))
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    return rank, world, local


def spawn_ranks(n_gpus: int) -> int:
    """Started without torchrun but with --gpus N > 1: run this very command line as N ranks of one
    node (rendezvous on 127.0.0.1, a free port) and return the launcher's exit code."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.call(cmd)


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()


def max_over_ranks(value: float, world: int, device) -> float:
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# ----------------------------------------------------------------------------
# the CPU oracle as a timed baseline (only this function touches oracle/)
# ----------------------------------------------------------------------------
def oracle_pass(case: wl.Case, act: str, x_np, g_np, tables, threads: int) -> float:
    """One pass of the hot path (all bit widths, forward + backward) through the
    oracle as it stands, the sample cut into `threads` shards on 32-element
    boundaries, one oracle call per shard.  Returns seconds."""
    import concurrent.futures

    import oracle

    n = x_np.size
    cuts = [wl.shard_range(n, r, threads, 1024) for r in range(threads)]

    def work(rng):
        lo, hi = rng
        for bits in case.bits:
            s, lev = tables[bits]
            _, p = oracle.fwd(act, bits, s, x_np[lo:hi])
            oracle.bwd(bits, lev, p, g_np[lo:hi])

    t0 = time.perf_counter()
    with concurrent.futures.ThreadPoolExecutor(max_workers=threads) as pool:
        list(pool.map(work, cuts))
    return time.perf_counter() - t0


def oracle_tables(case: wl.Case, act: str):
    import oracle
    import numpy as np

    out = {}
    for bits in case.bits:
        r = oracle.dp_solve(act, bits)
        out[bits] = (r["s"].astype(np.float32), r["lev"].astype(np.float32))
    return out


def cpu_baseline(case: wl.Case, act: str, sample_elems: int):
    import oracle  # noqa: F401  (builds the shared object outside the timed region)
    threads = len(os.sched_getaffinity(0))
    x, g = wl.draw(case, "cpu", n=sample_elems)
    x_np, g_np = wl.to_numpy_bits(x), wl.to_numpy_bits(g)
    tables = oracle_tables(case, act)
    secs = oracle_pass(case, act, x_np, g_np, tables, threads)
    passes = 2 * len(case.bits) * sample_elems
    # the same on one thread, on 1/16 of the sample (the oracle itself is single-threaded plain C)
    one = max(1024, sample_elems // 16)
    secs_one = oracle_pass(case, act, x_np[:one], g_np[:one], tables, 1)
    return {"value": passes / secs, "unit": "elements/s", "cores": threads, "kind": "oracle",
            "sample": f"first {sample_elems} elements of the {case.name} draw, bits {list(case.bits)}, fwd+bwd, "
                      f"{threads} shards on {threads} threads, {secs:.2f} s",
            "value_one_thread": 2 * len(case.bits) * one / secs_one,
            "sample_one_thread": f"first {one} elements, 1 thread, {secs_one:.2f} s"}


# ----------------------------------------------------------------------------
# reference arm: the oracle on host cores
# ----------------------------------------------------------------------------
def run_reference(args, case: wl.Case, act: str):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle  # noqa: F401
    threads = len(os.sched_getaffinity(0))
    sample = args.ref_sample
    x, g = wl.draw(case, "cpu", n=sample)
    x_np, g_np = wl.to_numpy_bits(x), wl.to_numpy_bits(g)
    tables = oracle_tables(case, act)
    for _ in range(args.warmup):
        oracle_pass(case, act, x_np, g_np, tables, threads)
    t = 0.0
    for _ in range(args.steps):
        t += oracle_pass(case, act, x_np, g_np, tables, threads)
    passes = 2 * len(case.bits) * sample * args.steps
    value = passes / t
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "elements/s", "n_gpus": args.gpus,
        "ranks_started": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": case.dtype, "data": "synthetic",
        "config": {"workload": case.name, "act": act, "bits": list(case.bits), "elements_per_step_sample": sample,
                   "note": "CPU oracle on a bounded sample of the workload; elements counted once per kernel-equivalent pass"},
        "cpu_baseline": {"value": value, "unit": "elements/s", "cores": threads, "kind": "oracle",
                         "sample": f"first {sample} elements of the {case.name} draw per step"},
        "e2e": {"value": value, "unit": "elements/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------
def run_ours(args, case: wl.Case, act: str):
    import paper_2202_00441_b200 as fb

    rank, world, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    fb.load_library()

    n_total = args.elements or case.n
    strong = args.scaling == "strong"
    if strong:
        # one tensor for the whole job (every rank draws it with the same seed), cut on multiples of
        # 32 elements: each shard's packed words are whole, no rank touches another's data
        xf, gf = wl.draw(case, dev, n=n_total)
        lo, hi = wl.shard_range(n_total, rank, world, align=32)
        x, g = xf[lo:hi].clone(), gf[lo:hi].clone()
        del xf, gf
        torch.cuda.empty_cache()
        n = hi - lo
    else:
        n = n_total
        x, g = wl.draw(dataclass_replace_seed(case, case.seed + rank), dev, n=n)
    y, gi = torch.empty_like(x), torch.empty_like(g)
    tables = {b: fb.fewbit_table_create(act, b) for b in case.bits}
    packed = {b: torch.empty(fb.fewbit_packed_bytes(n, b) // 4, dtype=torch.int32, device=dev) for b in case.bits}
    footprint = (x.numel() * x.element_size()) * 4 + sum(p.numel() * 4 for p in packed.values())
    # Smaller than a few L2s: L2-cold by rotation over copies of the buffers, a different copy for every
    # launch (a flush write would leave the L2 full of dirty lines whose write-back the next kernel pays).
    sets = 1 if footprint >= 512 * 2 ** 20 else int(512 * 2 ** 20 // footprint) + 2
    bufs = [(x, g, y, gi, packed)]
    for _ in range(sets - 1):
        bufs.append((x.clone(), g.clone(), torch.empty_like(y), torch.empty_like(gi), {b: torch.empty_like(p) for b, p in packed.items()}))
    if sets > 1:                              # a backward reads the words an earlier forward left in another copy
        for xs, _, ys, _, ps in bufs:
            for b in case.bits:
                fb.fewbit_fwd(tables[b], xs, ys, ps[b])

    order = [(kind, b) for b in case.bits for kind in ("fwd", "bwd")]
    turn = [0]

    def one_step(events=None):
        for i, (kind, b) in enumerate(order):
            xs, gs, ys, gis, ps = bufs[turn[0] % sets]
            turn[0] += 1
            if events is not None:
                events[i][0].record()
            if kind == "fwd":
                fb.fewbit_fwd(tables[b], xs, ys, ps[b])
            else:
                fb.fewbit_bwd(tables[b], ps[b], gs, gis)
            if events is not None:
                events[i][1].record()

    for _ in range(args.warmup):
        one_step()
    ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in order]
          for _ in range(args.steps)]
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    barrier(world)
    launches_before = fb.fewbit_launch_count()
    t_begin = time.time()
    if sets > 1:
        # launches of a few microseconds: a device-side delay ahead of the first event lets the host run
        # ahead, so that the events bracket GPU time and not the Python launch latency (~25 us a call)
        torch.cuda._sleep(min(int(args.steps * len(order) * 40e-6 * 2e9), 1 << 30))
    start.record()
    for s in range(args.steps):
        one_step(ev[s])
    stop.record()
    barrier(world)
    t_end = time.time()
    launches_in_region = fb.fewbit_launch_count() - launches_before
    clocks = sampler.stop(t_begin, t_end) if rank == 0 else None
    total_ms = start.elapsed_time(stop)
    total_ms = max_over_ranks(total_ms, world, dev)

    per_kernel = {}
    for i, (kind, b) in enumerate(order):
        ms = [ev[s][i][0].elapsed_time(ev[s][i][1]) for s in range(args.steps)]
        avg = sum(ms) / len(ms)
        by = algorithmic_bytes(case, n, b)
        per_kernel[f"{kind}_k{b}"] = {"avg_us": 1e3 * avg, "min_us": 1e3 * min(ms), "gbs": by / (avg * 1e-3) / 1e9,
                                      "gelems": n / (avg * 1e-3) / 1e9, "bytes": by}
    peak, peak_kind = measured_peak()
    dom = max(per_kernel, key=lambda k: per_kernel[k]["avg_us"])
    roofline = {"bound": "hbm", "kernel": dom, "achieved": per_kernel[dom]["gbs"], "peak": peak, "unit": "GB/s",
                "frac": per_kernel[dom]["gbs"] / peak, "peak_kind": f"of {peak_kind}",
                "frac_of_nominal_8TBs": per_kernel[dom]["gbs"] / NOMINAL_HBM_GBS,
                "traffic": NCU_TRAFFIC_BYTES_PER_ELEM.get((case.dtype, dom)) and
                NCU_TRAFFIC_BYTES_PER_ELEM[(case.dtype, dom)] * n}
    n_job = n_total if strong else world * n                   # elements all ranks process per kernel pass
    elems_per_step = 2 * len(case.bits) * n_job
    value = elems_per_step * args.steps / (total_ms * 1e-3)
    bytes_per_step = 2 * sum(algorithmic_bytes(case, n_job, b) for b in case.bits)
    # Sum over the bit patterns of every output of one step (y and grad_in of the last bit width, the
    # packed words of every width), added up over the ranks: with --scaling strong it does not depend on N.
    xs0, gs0, ys0, gis0, ps0 = bufs[0]
    iview = torch.int32 if case.dtype == "f32" else torch.int16
    checksum = 0
    for b in case.bits:
        fb.fewbit_fwd(tables[b], xs0, ys0, ps0[b])
        checksum += int(ps0[b].to(torch.int64).sum().item())
    fb.fewbit_bwd(tables[case.bits[-1]], ps0[case.bits[-1]], gs0, gis0)
    checksum += int(ys0.view(iview).to(torch.int64).sum().item()) + int(gis0.view(iview).to(torch.int64).sum().item())
    if world > 1:
        import torch.distributed as dist
        cs = torch.tensor([checksum], dtype=torch.int64, device=dev)
        dist.all_reduce(cs)
        checksum = int(cs.item())
    checksum &= (1 << 63) - 1

    # ---- end to end through the host-buffer entry points -----------------------------------------
    e2e = None
    if not args.no_e2e:
        hx, hg = x.cpu().pin_memory(), g.cpu().pin_memory()
        hy, hgi = torch.empty_like(hx).pin_memory(), torch.empty_like(hg).pin_memory()
        hp = {b: torch.empty(packed[b].numel(), dtype=torch.int32).pin_memory() for b in case.bits}
        ws = torch.empty(fb.fewbit_host_workspace_bytes(1 << 23, x.dtype, max(case.bits)), dtype=torch.uint8, device=dev)

        def e2e_step():
            for b in case.bits:
                fb.fewbit_fwd_host(tables[b], hx, hy, hp[b], ws)
                fb.fewbit_bwd_host(tables[b], hp[b], hg, hgi, ws)

        e2e_step()
        barrier(world)
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            e2e_step()
        barrier(world)
        secs = max_over_ranks(time.perf_counter() - t0, world, dev)
        eb = elem_size(case)
        h2d = sum(n * eb + (n * eb + packed[b].numel() * 4) for b in case.bits)
        d2h = sum((n * eb + packed[b].numel() * 4) + n * eb for b in case.bits)
        e2e = {"value": elems_per_step * args.e2e_steps / secs, "unit": "elements/s",
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": args.e2e_steps,
               "gbs_pcie_each_way": h2d * args.e2e_steps / secs / 1e9,
               "api": "fewbit_fwd_host / fewbit_bwd_host on pinned host tensors"}
        del hx, hg, hy, hgi, hp, ws

    # ---- plain unfused PyTorch activation (context) -----------------------------------------------
    torch_ref = None
    if rank == 0 and not args.no_torch_baseline:
        torch_ref = torch_unfused(case, act, x, g)

    # ---- the other configurations, quick device-resident runs (context) --------------------------
    also = {}
    if rank == 0 and not args.no_also:
        for name in ("c2", "c4", "c1"):
            if wl.CONFIGS[name].name != case.name:
                also[name] = quick_config(fb, wl.CONFIGS[name], dev)
        also["c4_folded"] = quick_config(fb, wl.C4, dev, folded=True)      # even-derivative fold: codes from |x|
        import dataclasses
        f16 = dataclasses.replace(wl.C3, name="c3_shape_f16_2p26", dtype="f16", shape=(1 << 26,), bits=(1, 4))
        also["f16"] = quick_config(fb, f16, dev, reps=5)                   # IEEE binary16 storage
        also["c2_bias"] = quick_config(fb, wl.C2, dev, bias_cols=wl.C2.shape[-1])   # f(x + bias), the add inside the kernel
        del x, g, y, gi, packed, bufs, xs0, gs0, ys0, gis0, ps0
        torch.cuda.empty_cache()
        also["c5"] = c5_summary(fb, dev, peak)                              # the sweep at >= 16 M elements, compact

    cpu = None
    if rank == 0 and not args.no_cpu_baseline:
        cpu = cpu_baseline(case, act, args.cpu_sample)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "elements/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": args.scaling,
            "vs_baseline": None, "dtype": case.dtype, "data": "synthetic",
            "config": {"workload": case.name if not args.elements else f"{case.name} cut to {n} elements",
                       "act": act, "bits": list(case.bits), "shape": list(case.shape) if not args.elements else [n_total],
                       "elements": n_job, "elements_per_rank": n, "launches_per_step": len(order),
                       "l2": "inputs larger than L2 (no flush)" if sets == 1 else f"cold by rotation over {sets} copies of the buffers ({sets * footprint / 2 ** 20:.0f} MiB), a different one every launch; launches queued behind a device-side delay",
                       "elements_counted": "once per kernel pass (forward and backward each count n)",
                       "parallelism": (f"one tensor cut into {world} shards on multiples of 32 elements" if strong
                                       else f"independent tensors x{world}") + ", no collective on the data path"},
            "checksum": checksum, "nccl_log": os.environ.get("NCCL_DEBUG_FILE") if world > 1 else None,
            "hbm_gbs": bytes_per_step * args.steps / (total_ms * 1e-3) / 1e9,
            "hbm_frac_of_nominal_8TBs": bytes_per_step * args.steps / (total_ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS / world,
            "hbm_frac_of_measured_copy": bytes_per_step * args.steps / (total_ms * 1e-3) / 1e9 / peak / world,
            "roofline": roofline, "kernels": per_kernel, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": launches_in_region, "clocks": clocks, "torch_unfused": torch_ref, "also": also,
            "saved_activation_ratio": {str(b): 8 * elem_size(case) / b for b in case.bits},
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# DRAM bytes per element (dram__bytes_read.sum + dram__bytes_write.sum of one launch / n) from the ncu
# captures of the 2^27-element launches of these kernels; None for a kernel without a capture.
NCU_TRAFFIC_BYTES_PER_ELEM = {
    # scaled per element: a lower bound for the full launch, the L2 keeps ~55 MB of dirty lines either way
    ("bf16", "fwd_k4"): 4.098,
    ("bf16", "bwd_k4"): 4.085,
    ("bf16", "fwd_k1"): 3.729,
}


def dataclass_replace_seed(case: wl.Case, seed: int) -> wl.Case:
    import dataclasses
    return dataclasses.replace(case, seed=seed)


def torch_unfused(case: wl.Case, act: str, x, g, reps: int = 5):
    import torch.nn.functional as F
    fn = {"gelu": F.gelu, "silu": F.silu, "sigmoid": torch.sigmoid, "tanh": torch.tanh, "elu": F.elu,
          "softplus": F.softplus, "leaky_relu": F.leaky_relu}[act]
    xr = x.detach().clone().requires_grad_(True)
    a, b, c = (torch.cuda.Event(enable_timing=True) for _ in range(3))
    fwd_ms, bwd_ms = [], []
    for i in range(reps + 2):
        a.record()
        out = fn(xr)
        b.record()
        out.backward(g)
        c.record()
        torch.cuda.synchronize()
        xr.grad = None
        if i >= 2:
            fwd_ms.append(a.elapsed_time(b)); bwd_ms.append(b.elapsed_time(c))
        del out
    n, eb = case.n, elem_size(case)
    return {"fwd_us": 1e3 * min(fwd_ms), "bwd_us": 1e3 * min(bwd_ms),
            "fwd_gbs": 2 * eb * n / (min(fwd_ms) * 1e-3) / 1e9, "bwd_gbs": 3 * eb * n / (min(bwd_ms) * 1e-3) / 1e9,
            "saved_bytes_per_elem": eb, "note": "stock torch forward + autograd backward, full input kept"}


def batch_median_ms(launch, inner: int, reps: int) -> float:
    """Median over `reps` timings (after 3 untimed ones) of a back-to-back batch of `inner` launches,
    per launch, in ms: launch(i, j) enqueues launch j of timing i.  A spin kernel ahead of the first
    event keeps the GPU busy (no memory traffic) while the host enqueues, so the events bracket GPU
    time, not launch latency."""
    ms = []
    for i in range(reps + 3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda._sleep(400000)
        e0.record()
        for j in range(inner):
            launch(i, j)
        e1.record()
        torch.cuda.synchronize()
        if i >= 3:
            ms.append(e0.elapsed_time(e1) / inner)
    return statistics.median(ms)


def quick_config(fb, case: wl.Case, dev, reps: int = 10, folded: bool = False, bias_cols: int = 0):
    """Device-resident timing of another configuration.  L2-cold by rotation: enough independent
    buffer sets that their footprint exceeds 4x the 126 MB L2, a different set for every launch
    (a write-flush would leave the L2 full of dirty lines whose write-back is then charged to a
    kernel that only runs for a few microseconds).  A spin kernel ahead of the first event lets the
    host finish enqueueing, so the events bracket GPU time, not launch latency.  bias_cols > 0: the
    forward is fewbit_fwd_bias with a bias of that many columns (f(x + bias), the add fused in)."""
    eb = elem_size(case)
    per_set = case.n * (4 * eb + 0.5)
    sets = max(2, int(512 * 2 ** 20 // per_set) + 1)
    if per_set < 512 * 2 ** 20:
        sets = max(sets, 9)
    # the event clock ticks every ~2 us: short kernels are timed as a back-to-back batch of up to 8
    # launches (launch gaps included), each on another buffer set
    inner = max(1, min(sets - 1, 8)) if per_set < 512 * 2 ** 20 else 1
    x0, g0 = wl.draw(case, dev)
    xs = [x0] + [x0.clone() for _ in range(sets - 1)]
    gs = [g0] + [g0.clone() for _ in range(sets - 1)]
    ys = [torch.empty_like(x0) for _ in range(sets)]
    gis = [torch.empty_like(g0) for _ in range(sets)]
    bias = torch.randn(bias_cols, device=dev).mul_(0.5).to(x0.dtype) if bias_cols else None
    out = {}
    for act in case.acts:
        if folded and act not in ("sigmoid", "tanh"):
            continue
        for b in case.bits:
            t = fb.fewbit_table_create_folded(act, b) if folded else fb.fewbit_table_create(act, b)
            ps = [torch.empty(fb.fewbit_packed_bytes(case.n, b) // 4, dtype=torch.int32, device=dev) for _ in range(sets)]

            def fwd(k):
                if bias is None:
                    fb.fewbit_fwd(t, xs[k], ys[k], ps[k])
                else:
                    fb.fewbit_fwd_bias(t, xs[k].view(-1, bias_cols), bias, ys[k], ps[k])

            # cold: a different buffer set every launch (the forward timings leave codes in every set)
            fm = batch_median_ms(lambda i, j: fwd((i * inner + j) % sets), inner, reps)
            bm = batch_median_ms(lambda i, j: fb.fewbit_bwd(t, ps[(i * inner + j) % sets], gs[(i * inner + j) % sets],
                                                            gis[(i * inner + j) % sets]), inner, reps)
            by = algorithmic_bytes(case, case.n, b)
            out[f"{act}_k{b}"] = {"fwd_us": 1e3 * fm, "bwd_us": 1e3 * bm, "fwd_gbs": by / (fm * 1e-3) / 1e9,
                                  "bwd_gbs": by / (bm * 1e-3) / 1e9}
            if case.n * (2 * eb + 0.5) < 100 * 2 ** 20:
                # L2-warm, labelled as such: the same buffers again and again (what one kernel touches fits the 126 MB L2)
                warm = max(inner, 8)
                out[f"{act}_k{b}"]["fwd_us_l2_warm"] = 1e3 * batch_median_ms(lambda i, j: fwd(0), warm, reps)
                out[f"{act}_k{b}"]["bwd_us_l2_warm"] = 1e3 * batch_median_ms(lambda i, j: fb.fewbit_bwd(t, ps[0], gs[0], gis[0]), warm, reps)
    return {"workload": case.name, "elements": case.n, "dtype": case.dtype,
            "l2": f"cold by rotation over {sets} buffer sets ({sets * per_set / 2 ** 20:.0f} MiB)",
            "launches_per_timing": inner, "cases": out}


def c5_summary(fb, dev, peak: float, sizes=(2 ** 24, 2 ** 24 + 7, 2 ** 28), reps: int = 3):
    """Config 5 at the sizes of at least 16 M elements, compact: per size and dtype, for every bit
    width the minimum and the median over the seven activations of the forward and backward fraction
    of the copy bandwidth (`peak`), the activation with the slowest forward, and what a torch copy_
    with the traffic of the 2-bit kernels reaches at that size, timed the same way."""
    out = {}
    for case in wl.sweep_cases(sizes):
        r = quick_config(fb, case, dev, reps=reps)["cases"]
        row = {"copy_same_traffic_frac": round(copy_at_size(int(algorithmic_bytes(case, case.n, 2)) // 2, dev, reps=reps) / peak, 3)}
        for kind in ("fwd", "bwd"):
            per_bits = [[r[f"{a}_k{b}"][f"{kind}_gbs"] / peak for a in case.acts] for b in case.bits]
            row[f"{kind}_frac_min"] = [round(min(v), 3) for v in per_bits]
            row[f"{kind}_frac_median"] = [round(statistics.median(v), 3) for v in per_bits]
        row["slowest_fwd"] = [min(case.acts, key=lambda a: r[f"{a}_k{b}"]["fwd_gbs"]) for b in case.bits]
        out[f"{case.dtype}_{case.n}"] = row
        torch.cuda.empty_cache()
    return {"bits": [1, 2, 3, 4], "activations": list(wl.ACTIVATIONS), "frac_of": f"{peak} GB/s", "cases": out}


def copy_at_size(nbytes: int, dev, reps: int = 10):
    """GB/s of a torch copy_ that reads nbytes and writes nbytes, timed like quick_config (L2-cold by
    rotation, short launches as a back-to-back batch): what a plain copy reaches at a given size."""
    sets = max(2, (512 << 20) // (2 * nbytes) + 1)
    if 4 * nbytes < (512 << 20):
        sets = max(sets, 9)
    inner = max(1, min(sets - 1, 8)) if 4 * nbytes < (512 << 20) else 1
    src = [torch.zeros(nbytes, dtype=torch.uint8, device=dev) for _ in range(sets)]
    dst = [torch.empty(nbytes, dtype=torch.uint8, device=dev) for _ in range(sets)]
    ms = batch_median_ms(lambda i, j: dst[(i * inner + j) % sets].copy_(src[(i * inner + j) % sets]), inner, reps)
    return 2 * nbytes / (ms * 1e-3) / 1e9


def run_sweep(args):
    """The size / activation / width / dtype sweep (config 5): one JSON line with the forward and backward
    time of every case and the fraction of the measured copy bandwidth each reaches (the 2^16 and 2^20
    points are launch-bound: read their times, not their fractions).  A context run on one GPU, not the
    contract line."""
    import paper_2202_00441_b200 as fb
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, peak_kind = measured_peak()
    out = {}
    for case in wl.sweep_cases():
        if args.act:
            case = dataclasses.replace(case, acts=(args.act,))
        r = quick_config(fb, case, dev, reps=7)
        for c in r["cases"].values():
            c["fwd_frac"], c["bwd_frac"] = c["fwd_gbs"] / peak, c["bwd_gbs"] / peak
        # a plain copy with the traffic of the 2-bit kernels of this size, for scale
        r["torch_copy_same_traffic_frac"] = copy_at_size(int(algorithmic_bytes(case, case.n, 2)) // 2, dev) / peak
        out[case.name] = r
        torch.cuda.empty_cache()
    print(json.dumps({"sweep": "c5", "peak_gbs": peak, "peak_kind": f"of {peak_kind}", "cases": out}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--scaling", choices=["weak", "strong"], default="weak",
                    help="N > 1: weak = a tensor of the workload per rank; strong = one tensor cut into N shards")
    ap.add_argument("--workload", choices=sorted(wl.CONFIGS), default="c3")
    ap.add_argument("--act", default=None, help="activation of the workload to time (default: its first)")
    ap.add_argument("--bits", default=None, help="comma-separated bit widths instead of the workload's own (profiling aid)")
    ap.add_argument("--elements", type=int, default=0,
                    help="draw only this many elements of the workload's distribution (small cases for profiling)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--cpu-sample", type=int, default=1 << 26)
    ap.add_argument("--ref-sample", type=int, default=1 << 25)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-torch-baseline", action="store_true")
    ap.add_argument("--no-also", action="store_true")
    ap.add_argument("--sweep", action="store_true",
                    help="time config 5 (7 activations x 1-4 bits x bf16/fp32 at 2^16, 2^20, 2^24, 2^24+7 and 2^28 elements) instead")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(spawn_ranks(args.gpus))
    if args.sweep:
        return run_sweep(args)
    args.warmup = max(args.warmup, 0)
    case = wl.CONFIGS[args.workload]
    if args.bits:
        case = dataclasses.replace(case, name=f"{case.name} at bits {args.bits}", bits=tuple(int(b) for b in args.bits.split(",")))
    act = args.act or case.acts[0]
    if args.impl == "reference":
        run_reference(args, case, act)
    else:
        run_ours(args, case, act)


if __name__ == "__main__":
    main()
