#!/usr/bin/env python
"""Benchmark of the DoubleSqueeze step (worker pass + server pass with fused model update).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1..12] [--impl ours|reference]

One "step" is one whole iteration of Algorithm 1 over one batch of synthetic gradients
(ds_worker_compress + ds_server_aggregate_compress with the fused update).  Prints ONE JSON line.

Without --workload the five listed configurations are all measured in one run; the headline keys
(value, ms_per_step, roofline, e2e, cpu_baseline, config) are those of the largest one, workload 5
(32 workers x 60 M entries, 1-bit workers, top-k server with the paper's k = 300000), and
"per_workload" carries the record of each.  With --workload N only that one is run.

A workload is timed in blocks of K steps (CUDA events on the launching stream); blocks are repeated
until at least --min-seconds of GPU time are in, and the median block gives the headline, the
spread over blocks and over steps is reported beside it.

For N > 1 (launched by torch.distributed.run) every rank steps an independent replica of the same
workloads on its own GPU -- the path has no exchange between GPUs -- and the value is the aggregate.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "doublesqueeze_step_gradient_elements_per_s"
UNIT = "elements/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
LISTED = (1, 2, 3, 4, 5)     # the five listed configurations
HEADLINE = 5                 # the largest one that fits one GPU

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# captures summarised under profiles/; valid only for the kernel sources with this digest.
# (kernel, bytes in the captured launch, gradient entries the captured launch processed, digest of
# the kernel's source files at capture time).  A capture taken at a smaller size than the workload
# (a multi-pass capture must stay small) is scaled by the entries one launch processes: the
# traffic of a streaming kernel grows in proportion.
NCU_CAPTURES = {
    "sign1": ("k_chunked<SIGN1, WORKER, 4, 256>", 748182272 + 331582464, 8 * 11_689_512, "3e80faecea9d3b0a"),
    "qsgd": ("k_chunked<QSGD, WORKER, 2, 256>", 1073773000 + 630182144, 8 * 16_777_216, "3e80faecea9d3b0a"),
    # the first kernel of the top-k worker pass alone (v read once, written once); the selection that follows it
    # moves a few percent of that
    "topk": ("k_topk_pass1<WORKER>", 537251328 + 221441280, 16 * 4_194_304, "8493784d4c9f8058"),
    "clip": ("k_clip<WORKER, 16>", 748323328 + 508980736, 8 * 11_689_512, "ccfe82e0a4de6e6b"),
    "rsparse": ("k_rsparse<WORKER>", 748263680 + 333547008, 8 * 11_689_512, "ccfe82e0a4de6e6b"),
}
KERNEL_SOURCES = {  # files whose change invalidates the captured counters
    "sign1": ("dsq_chunked.cuh", "dsq_common.cuh", "dsq_internal.h"),
    "qsgd": ("dsq_chunked.cuh", "dsq_common.cuh", "dsq_internal.h"),
    "topk": ("dsq_topk.cu", "dsq_common.cuh", "dsq_internal.h"),
    "identity": ("dsq_elementwise.cu", "dsq_common.cuh", "dsq_internal.h"),
    "clip": ("dsq_elementwise.cu", "dsq_common.cuh", "dsq_internal.h"),
    "rsparse": ("dsq_elementwise.cu", "dsq_common.cuh", "dsq_internal.h"),
    "ternary": ("dsq_whole.cu", "dsq_chunked.cuh", "dsq_common.cuh", "dsq_internal.h"),
}
DOMINANT = {"ternary": "k_whole_reduce / k_whole_ternary_draw / k_whole_ternary_apply <WORKER>", "sign1": "k_chunked<SIGN1, WORKER>", "qsgd": "k_chunked<QSGD, WORKER>",
            "topk": "top-k worker pass (k_topk_pass1<WORKER> and the selection tail)",
            "identity": "k_identity<WORKER>", "clip": "k_clip<WORKER>", "rsparse": "k_rsparse<WORKER>"}


def payload_bytes(q, d: int) -> int:
    nw = (d + 31) // 32
    if q.op == "sign1":
        return 4 * nw + 4 * ((d + q.chunk - 1) // q.chunk if q.chunk else 1)
    if q.op == "qsgd":
        return d + 4 * nw + 4 * ((d + q.chunk - 1) // q.chunk)
    if q.op == "topk":
        return 8 * q.k
    if q.op == "clip":
        return d * (32 - q.bits) // 8
    if q.op == "rsparse":
        nc = (d + q.chunk - 1) // q.chunk
        return 4 * nc * (q.chunk // q.keep_one_in) + 4 * nc
    if q.op == "ternary":
        return 8 * nw + 4
    return 4 * d


def algorithmic_bytes(wl) -> dict:
    """Bytes the method must move per step: read g and delta_w, write delta_w and the worker
    payloads; the server reads the payloads, reads and writes delta_s, writes its payload, and
    reads and writes x (only the k kept entries for top-k)."""
    n, d = wl.n, wl.d
    pw, ps = payload_bytes(wl.worker_q, d), payload_bytes(wl.server_q, d)
    err = 8 if wl.compensate else 0          # an error is read and written, or there is none
    worker = n * d * (4 + err) + n * pw
    x_bytes = 8 * wl.server_q.k if wl.server_q.op == "topk" else 8 * d
    server = n * pw + err * d + ps + x_bytes
    return {"worker": worker, "server": server, "total": worker + server}


def csrc_digest(op: str) -> str:
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_1905_05957_b200", "csrc")
    for f in KERNEL_SOURCES[op]:
        h.update(open(os.path.join(csrc, f), "rb").read())
    return h.hexdigest()[:16]


def captured_traffic(wl):
    """DRAM bytes per launch of the workload's dominant kernel from the committed capture, scaled to
    this launch's entries; None without a capture or once the kernel's sources have changed."""
    cap = NCU_CAPTURES.get(wl.worker_q.op)
    whole = wl.worker_q.op == "sign1" and wl.worker_q.chunk == 0     # other kernels than the captured ones
    if cap is None or whole or not wl.compensate or cap[3] != csrc_digest(wl.worker_q.op):
        return None
    return int(cap[1] * (wl.n * wl.d) / cap[2])


def measured_peak() -> tuple[float, str]:
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def pct(xs, q: float) -> float:
    s = sorted(xs)
    return s[int(q * (len(s) - 1))]


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def wait_first(self, seconds: float = 3.0):
        """The first answer takes a moment; what came before the load is dropped."""
        t_wait = time.time() + seconds
        while self.proc is not None and not self.lines and time.time() < t_wait:
            time.sleep(0.05)
        self.lines.clear()

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx = float(parts[1])
            except ValueError:
                continue
            for nm, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ---------------------------------------------------------------------------------------------
# reference arm and CPU baseline: the oracle, as it stands, on the host cores
# ---------------------------------------------------------------------------------------------

# rough single-thread cost of the oracle per vector entry (seconds), used only to size the sample
ORACLE_COST = {"identity": 0.6e-8, "sign1": 1.2e-8, "qsgd": 3.0e-8, "topk": 1.3e-7, "clip": 0.8e-8, "rsparse": 0.8e-8,
               "ternary": 3.0e-8}


def oracle_sample_workload(wl, seconds_per_step: float):
    """A bounded sample of the workload for the CPU oracle: same recipe and n workers, d cut so that
    one step is about `seconds_per_step` of single-thread work."""
    per_d = wl.n * (ORACLE_COST.get(wl.worker_q.op, 3e-8) + 1.0e-8) + ORACLE_COST.get(wl.server_q.op, 3e-8) + 1.0e-8
    d = int(seconds_per_step / per_d)
    if d >= wl.d:
        return wl, "full workload"
    d = max(8192, d // 8192 * 8192)
    return wl.scaled(d=d), f"same recipe with d cut to {d} (n={wl.n})"


def time_oracle(wl, steps: int, warmup: int, seconds_per_step: float) -> dict:
    import numpy as np

    import oracle
    from paper_1905_05957_b200.workloads import make_gradients

    swl, what = oracle_sample_workload(wl, seconds_per_step)
    st = oracle.State.zeros(swl.n, swl.d)
    wq, sq = oracle.qspec_from(swl.worker_q), oracle.qspec_from(swl.server_q)
    gs = [make_gradients(swl, t, device="cpu").numpy() for t in range(2)]
    for t in range(warmup):
        oracle.step(st, gs[t % 2], wq, sq, swl.gamma, swl.seed, t, compensate=swl.compensate)
    t0 = time.perf_counter()
    for t in range(steps):
        oracle.step(st, gs[t % 2], wq, sq, swl.gamma, swl.seed, warmup + t, compensate=swl.compensate)
    dt = time.perf_counter() - t0
    assert np.isfinite(st.x).all()
    return {"value": swl.n * swl.d * steps / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{steps} step(s) of {what}; single thread", "ms_per_step": 1e3 * dt / steps}


def run_reference(args, wl):
    """The reference arm: the oracle, as it stands, for exactly --steps timed steps after --warmup
    untimed ones; the sample of the workload is sized so that the whole run takes about two and a
    half minutes whatever K and W are."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    per_step = min(5.0, 150.0 / (steps + warmup))
    r = time_oracle(wl, steps, warmup, per_step)
    line = {
        "impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": r["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(wl),
        "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
        "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(wl) -> dict:
    def q(s):
        return {"op": s.op, **({"chunk": s.chunk} if s.chunk else {}), **({"k": s.k} if s.op == "topk" else {}),
                **({"levels": s.levels} if s.levels else {}), **({"norm": "l2"} if s.op == "sign1" and s.norm == 2 else {}),
                **({"bits_cleared": s.bits} if s.op == "clip" else {}),
                **({"keep_one_in": s.keep_one_in, "scaled": bool(s.scaled)} if s.op == "rsparse" else {})}
    return {"workload": wl.name, "n_workers": wl.n, "d": wl.d, "gradient_dist": wl.dist, "worker_q": q(wl.worker_q),
            "server_q": q(wl.server_q), "gamma": wl.gamma, "error_compensation": wl.compensate,
            "l2": "inputs larger than L2: g and delta_w are streamed once per step and exceed 126 MB"
                  if wl.n * wl.d * 8 > 2 * 126e6 else "L2 flushed between steps by writing a 256 MB buffer"}


# ---------------------------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------------------------

class Env:
    def __init__(self):
        import torch
        import torch.distributed as dist
        self.torch, self.dist = torch, dist
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        if self.world > 1:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            dist.init_process_group("nccl")
        torch.cuda.set_device(self.local)
        self.dev = torch.device("cuda", self.local)

    def barrier(self):
        if self.world > 1:
            self.dist.barrier()
        self.torch.cuda.synchronize(self.dev)


def measure_workload(env: Env, wl, args, lib, want_e2e: bool) -> dict:
    """Times one workload on this rank's GPU; rank 0 gets the record."""
    torch = env.torch
    from paper_1905_05957_b200 import DoubleSqueeze
    from paper_1905_05957_b200.replicas import aggregate_throughput, max_over_ranks
    from paper_1905_05957_b200.workloads import make_gradients

    dev, world, rank = env.dev, env.world, env.rank
    K, W = args.steps, max(args.warmup, 3)
    ds = DoubleSqueeze.for_workload(wl, dev)
    # distinct g_t resident in HBM: a fresh draw for every step of a block where 100 GB hold them, else
    # a ring of as many as fit.  A training run never sees the same gradient twice, and a replayed
    # sequence makes the error feedback -- hence the top-k threshold -- follow the ring's period, so
    # where a threshold history matters the ring is drawn afresh (untimed) before every block.
    R = max(2, min(K + W, int(100e9 // (wl.n * wl.d * 4))))
    ring = [make_gradients(wl, t, device=dev) for t in range(R)]
    redraw = "topk" in (wl.worker_q.op, wl.server_q.op)
    drawn = R
    need_flush = wl.n * wl.d * 8 <= 2 * 126e6
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if need_flush else None
    stream = torch.cuda.current_stream(dev)
    E = lambda: torch.cuda.Event(enable_timing=True)

    step_no = 0
    for _ in range(W):
        ds.step(ring[step_no % R], step_no)
        step_no += 1
    sampler = ClockSampler(env.local)
    env.barrier()
    if rank == 0:
        sampler.start()
        sampler.wait_first()
    launches0 = lib.ds_kernel_launches()

    def timed_block():
        """EXACTLY K steps between a barrier + synchronize on both sides; returns the block's events."""
        nonlocal step_no
        ev = [[E() for _ in range(3)] for _ in range(K)]
        start, stop = E(), E()
        env.barrier()
        start.record(stream)
        for t in range(K):
            if need_flush:
                flush.fill_(t & 0xFF)
            ev[t][0].record(stream)
            ds.worker_compress(ring[step_no % R], step_no)
            ev[t][1].record(stream)
            ds.server_aggregate_compress(step_no, fuse_apply=True)
            ev[t][2].record(stream)
            step_no += 1
        stop.record(stream)
        env.barrier()
        steps = [(e[0].elapsed_time(e[1]), e[1].elapsed_time(e[2])) for e in ev]
        # the flush writes are not part of a step: with them the block is the sum of its steps
        total = sum(a + b for a, b in steps) if need_flush else start.elapsed_time(stop)
        return total, steps

    blocks, steps_all = [], []
    total, steps = timed_block()
    blocks.append(total)
    steps_all += steps
    # repeat the block until enough GPU time is in (every rank takes the same count)
    (slowest,) = max_over_ranks([total], device=dev)
    more = min(args.max_blocks, math.ceil(args.min_seconds * 1e3 / max(slowest, 1e-3))) - 1
    for _ in range(max(0, more)):
        if redraw:
            for slot in range(R):
                make_gradients(wl, drawn, device=dev, out=ring[slot])
                drawn += 1
        total, steps = timed_block()
        blocks.append(total)
        steps_all += steps
    launches = lib.ds_kernel_launches() - launches0
    # nvidia-smi answers every 100 ms: keep the same steps running, untimed, until a few samples under
    # this load are in
    t_end = time.time() + 1.2
    extra = 0
    while time.time() < t_end and (rank != 0 or len(sampler.lines) < 8):
        ds.step(ring[step_no % R], step_no)
        step_no += 1
        extra += 1
        if extra % 16 == 0:
            torch.cuda.synchronize(dev)
    torch.cuda.synchronize(dev)
    clocks = sampler.stop() if rank == 0 else None
    if clocks is not None:
        clocks["sampled"] = "during the timed blocks" + (" and the same steps repeated untimed right after them" if extra else "")
    status = ds.device_status()
    routes = ds.topk_routes()

    # ---- launch-bound workloads: the same step replayed from a CUDA graph (one graph per ring slot)
    graph_ms = None
    if need_flush:
        try:
            graphs = []
            for slot in range(2):
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr):
                    ds.step(ring[slot], 0)
                graphs.append(gr)
            stream = torch.cuda.current_stream(dev)
            gev = [[E() for _ in range(2)] for _ in range(K)]
            for t in range(3):
                graphs[t % 2].replay()
            env.barrier()
            for t in range(K):
                flush.fill_(t & 0xFF)
                gev[t][0].record(stream)
                graphs[t % 2].replay()
                gev[t][1].record(stream)
            env.barrier()
            graph_ms = statistics.median(gev[t][0].elapsed_time(gev[t][1]) for t in range(K))
        except Exception as exc:  # the number is an extra; the run does not depend on it
            graph_ms = f"unavailable: {type(exc).__name__}"

    # ---- end to end: pinned host g -> device, fused step, server payload -> host, every step
    e2e = None
    if want_e2e:
        big = wl.n * wl.d * 4 > 4e9     # pinning several GB takes seconds: one host buffer is enough there
        g_host = [torch.empty(wl.n, wl.d, dtype=torch.float32, pin_memory=True) for _ in range(1 if big else 2)]
        for a, b in zip(g_host, ring):
            a.copy_(b)
        out_host = torch.empty(ds.server_payload.numel(), dtype=torch.uint8, pin_memory=True)
        Ke = max(1, min(K, 10))
        for t in range(2):
            ds.step_host(g_host[t % len(g_host)], ring[0], 10_000_000 + t, server_payload_host=out_host)
        env.barrier()
        e0, e1 = E(), E()
        e0.record(stream)
        for t in range(Ke):
            ds.step_host(g_host[t % len(g_host)], ring[0], 20_000_000 + t, server_payload_host=out_host)
        e1.record(stream)
        env.barrier()
        (e2e_ms,) = max_over_ranks([e0.elapsed_time(e1)], device=dev)
        e2e = {"value": aggregate_throughput(wl.n * wl.d, Ke, e2e_ms, world), "unit": UNIT,
               "h2d_bytes_per_step": wl.n * wl.d * 4, "d2h_bytes_per_step": int(ds.server_payload.numel()), "steps": Ke}
        del g_host, out_host

    block_med = statistics.median(blocks)
    (block_med_slowest,) = max_over_ranks([block_med], device=dev)
    ds.close()
    del ds, ring, flush
    torch.cuda.empty_cache()
    if rank != 0:
        return {}

    ab = algorithmic_bytes(wl)
    peak, peak_kind = measured_peak()
    worker_ms = [a for a, _ in steps_all]
    server_ms = [b for _, b in steps_all]
    step_ms = [a + b for a, b in steps_all]
    wk_ms = statistics.mean(worker_ms)
    achieved = ab["worker"] / (wk_ms * 1e-3) / 1e9
    traffic = captured_traffic(wl)
    ms_per_step = block_med_slowest / K
    step_gbs = ab["total"] / (ms_per_step * 1e-3) / 1e9
    dominant = DOMINANT[wl.worker_q.op]
    if wl.worker_q.op == "sign1" and wl.worker_q.chunk == 0:
        dominant = "k_whole_reduce / k_whole_sign <WORKER>"
    roof = {"bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "peak_source": f"of {peak_kind}", "traffic": traffic,
            "algorithmic_bytes_per_launch": ab["worker"], "ms_per_launch": wk_ms,
            "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS,
            "dram_gbs_from_traffic": None if traffic is None else traffic / (wk_ms * 1e-3) / 1e9}
    if roof["frac"] > 1.0:
        roof["note"] = ("above 1: the peak is a plain device copy (read + write), not a hardware bound; this kernel reads "
                        "two bytes for every byte it writes, and reads run faster than writes")
    rec = {
        "workload": wl.name, "wid": wl.wid, "n_workers": wl.n, "d": wl.d,
        "ms_per_step": ms_per_step, "value": aggregate_throughput(wl.n * wl.d, K, block_med_slowest, world),
        "blocks": len(blocks), "steps_per_block": K, "gpu_seconds_timed": sum(blocks) * 1e-3,
        "block_ms_per_step": {"median": block_med / K, "p10": pct(blocks, 0.1) / K, "p90": pct(blocks, 0.9) / K},
        "step_ms": {"median": statistics.median(step_ms), "p10": pct(step_ms, 0.1), "p90": pct(step_ms, 0.9)},
        "worker_ms": wk_ms, "server_ms": statistics.mean(server_ms),
        "algorithmic_bytes": ab, "step_gbs": step_gbs,
        "step_frac_of_measured": step_gbs / peak, "step_frac_of_nominal_8000": step_gbs / NOMINAL_HBM_GBS,
        "server_gbs": ab["server"] / (statistics.mean(server_ms) * 1e-3) / 1e9,
        "roofline": roof, "clocks": clocks,
        "ms_per_step_x_sm_mhz": None if not clocks or not clocks.get("sm_mhz") else ms_per_step * clocks["sm_mhz"],
        "device_status": status, "gpu_launches": int(launches),
        "topk_routes": {"predicted": routes[0], "full": routes[1]},
    }
    if need_flush:
        rec["note"] = "launch-bound (a few MB per step): reported, not graded as a fraction of HBM bandwidth"
        rec["cuda_graph_step_ms_median"] = graph_ms
    if e2e is not None:
        rec["e2e"] = e2e
    if args.dump_steps:
        rec["step_ms_all"] = [round(x, 4) for x in step_ms]
    return rec


def run_ours(args, wids, headline):
    from paper_1905_05957_b200 import load_library
    from paper_1905_05957_b200.workloads import WORKLOADS

    env = Env()
    lib = load_library()          # raises if the CUDA library is missing: there is no other path
    recs = {}
    for wid in wids:
        wl = WORKLOADS[wid]
        if args.scale_d:
            wl = wl.scaled(d=args.scale_d)
        recs[wid] = measure_workload(env, wl, args, lib, want_e2e=(wid == headline))
    if env.rank == 0:
        wl = WORKLOADS[headline] if not args.scale_d else WORKLOADS[headline].scaled(d=args.scale_d)
        h = recs[headline]
        line = {
            "metric": METRIC, "value": h["value"], "unit": UNIT, "n_gpus": env.world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": h["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": workload_config(wl),
            "timing": f"median of {h['blocks']} blocks of {args.steps} steps each ({h['gpu_seconds_timed']:.2f} s of GPU time); "
                      "per_workload gives the spread",
            "clocks": h["clocks"], "e2e": h.get("e2e"), "gpu_launches": sum(r["gpu_launches"] for r in recs.values()),
            "roofline": h["roofline"],
            "step_frac_of_measured": h["step_frac_of_measured"], "step_frac_of_nominal_8000": h["step_frac_of_nominal_8000"],
            "device_status": max(r["device_status"] for r in recs.values()),
            "per_workload": [recs[w] for w in wids],
        }
        if not args.no_cpu_baseline and env.world == 1:
            r = time_oracle(wl, args.cpu_steps, 0, 5.0)
            line["cpu_baseline"] = {k: v for k, v in r.items() if k != "ms_per_step"}
        print(json.dumps(line), flush=True)
    if env.world > 1:
        env.dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------
# extra mode: one worker per GPU, server sharded over the GPUs (not the headline configuration)
# ---------------------------------------------------------------------------------------------

def run_sharded(args, wl):
    """Every rank is one worker (n = world size) and one slice of the server; the two compressed
    hops go over NCCL point-to-point operations.  Same timing rules as the default mode; the line
    says "mode": "sharded" and its value counts the n * d entries of one iteration."""
    import torch
    import torch.distributed as dist

    from paper_1905_05957_b200 import DoubleSqueeze, load_library
    from paper_1905_05957_b200.replicas import max_over_ranks
    from paper_1905_05957_b200.sharded import DistTransport, ShardedDoubleSqueeze
    from paper_1905_05957_b200.workloads import make_worker_gradient

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29517")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    lib = load_library()
    K, W = args.steps, max(args.warmup, 3)
    swl = wl.scaled(d=wl.d, n=world)
    # every rank keeps the error of its own worker only
    ds = DoubleSqueeze(world, swl.d, swl.gamma, swl.worker_q, swl.server_q, swl.seed, device=dev,
                       delta_w_rows=1 if world > 1 else 0)
    sh = ShardedDoubleSqueeze(ds, rank, world)
    tr = DistTransport()
    R = max(2, min(K + W, int(8e9 // (swl.d * 4))))
    ring = [make_worker_gradient(swl, t, rank, device=dev) for t in range(R)]
    stream = torch.cuda.current_stream(dev)

    def barrier():
        dist.barrier()
        torch.cuda.synchronize(dev)

    for t in range(W):
        sh.step(ring[t % R], t, tr)
    barrier()
    launches0 = lib.ds_kernel_launches()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for t in range(K):
        sh.step(ring[(W + t) % R], W + t, tr)
    e1.record(stream)
    barrier()
    (ms,) = max_over_ranks([e0.elapsed_time(e1)], device=dev)
    if rank == 0:
        line = {"metric": METRIC, "mode": "sharded", "value": world * swl.d * K / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
                "steps": K, "warmup": W, "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {**workload_config(swl), "workload": swl.name + "_one_worker_per_gpu", "n_workers": world},
                "gpu_launches": int(lib.ds_kernel_launches() - launches0), "device_status": ds.device_status()}
        print(json.dumps(line), flush=True)
    ds.close()
    dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50, help="steps per timed block")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", type=int, default=0,
                    help="0 (default): the five listed configurations in one run, headline = workload 5; 1..5 = one of them; "
                         "6..12 = shape of 2 with the l2-magnitude 1-bit scale / 16-bit clipping / randomised sparsification / "
                         "ternary quantiser / 1-bit with one factor per vector / the two methods without compensation")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--mode", default="replicas", choices=["replicas", "sharded"],
                    help="replicas (default): the listed single-GPU configuration on every GPU; sharded: one worker "
                         "per GPU with the server sharded over the GPUs (an extra, not the headline)")
    ap.add_argument("--min-seconds", type=float, default=0.5, help="GPU time to collect per workload (blocks are repeated)")
    ap.add_argument("--max-blocks", type=int, default=40)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-steps", type=int, default=5, help="oracle steps timed for cpu_baseline (about 2.3 s each on the headline sample)")
    ap.add_argument("--dump-steps", action="store_true", help="add the per-step times to the JSON line")
    ap.add_argument("--scale-d", type=int, default=0, help="run the workload's recipe at this d (profiling captures)")
    args = ap.parse_args()
    from paper_1905_05957_b200.workloads import WORKLOADS
    headline = args.workload or HEADLINE
    wids = (args.workload,) if args.workload else LISTED
    wl = WORKLOADS[headline]
    if args.scale_d:
        wl = wl.scaled(d=args.scale_d)
    if args.impl == "reference":
        run_reference(args, wl)
    elif args.mode == "sharded":
        run_sharded(args, wl)
    else:
        run_ours(args, wids, headline)


if __name__ == "__main__":
    main()
