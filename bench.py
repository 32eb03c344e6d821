#!/usr/bin/env python
"""Benchmark of the TOVA decode path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--capacity C]
  python bench.py --impl reference ...        # the CPU checker, timed on the host cores

A "step" is one decode step of one layer for the whole batch: split-K
attention over the full bounded state, combine, TOVA eviction and in-place
insert.  Steps rotate over enough independent layer caches that the working
set exceeds the L2 cache, the way the layers of a model follow each other.
Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "tova_decode_tokens_per_s_per_layer"
UNIT = "tokens/s"
RING = 128                      # distinct pre-generated tokens per workload
WORKING_SET = 1 << 30           # rotate layer caches until this many bytes are touched per round
# The largest single-GPU configuration: 32 layers of the LLaMA-2-7B shape, batch 64, state of 1024 rows
# (32 layer caches of 1 GiB; a step is one layer-step).
DEFAULT_WORKLOAD = "llama2_7b_full"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64, help="K: steps per timed unit (one CUDA graph of K steps)")
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--repeats", type=int, default=0,
                    help="how often the K timed steps are repeated (0 = until the timed region lasts 50 ms)")
    ap.add_argument("--no-sweep", action="store_true",
                    help="time the headline workload only, not the other graded configurations after it")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--capacity", type=int, default=0)
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--layers", type=int, default=0, help="independent layer caches to rotate over (0 = auto)")
    ap.add_argument("--chunk-rows", type=int, default=0)
    ap.add_argument("--no-graph", action="store_true", help="launch every step from the host instead of CUDA graphs")
    ap.add_argument("--policy", choices=["tova", "window", "tova_head", "h2o_layer", "h2o_head"], default="tova",
                    help="which row is dropped once the state is over capacity")
    ap.add_argument("--keep-first", type=int, default=0,
                    help="the +i of Window+i / TOVA+i; under H2O the size of the recent window (0 = half the state)")
    ap.add_argument("--position-compression", type=float, default=0.0, metavar="BASE",
                    help="time the position-compression mode (rotary embedding applied by the library with the "
                         "compressed positions); BASE = rotary base, e.g. 10000")
    ap.add_argument("--no-fused-merge", action="store_true",
                    help="merge the chunk partials through global memory even where a cluster could")
    ap.add_argument("--deferred", action="store_true", help="force deferred eviction on")
    ap.add_argument("--no-deferred", action="store_true",
                    help="pick the victim on the caller's stream instead of overlapping it with the next layer's step")
    ap.add_argument("--prefill", type=int, default=0, metavar="T",
                    help="time tova_prefill of a T-token prompt into an empty state instead of decode steps "
                         "(-1: as many tokens as the state holds); a step is one whole prompt")
    ap.add_argument("--no-bulk-prefill", action="store_true", help="with --prefill: every prompt token takes the decode kernels")
    ap.add_argument("--warp-mma-prefill", action="store_true", help="with --prefill: bulk fill through the warp-level MMA kernel")
    ap.add_argument("--chunk-barriers", type=int, default=0, choices=[0, 2],
                    help="with --prefill: 2 = the deletion kernel's cluster meets twice per token (0 = once where it fits)")
    ap.add_argument("--chunk-cluster", type=int, default=0,
                    help="with --prefill: thread blocks per sequence in the kernel that replays a chunk's deletions (0 = auto)")
    ap.add_argument("--no-chunked-prefill", action="store_true",
                    help="with --prefill: prompt tokens that meet a full state go one at a time instead of in chunks of 64")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    return ap.parse_args()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def pick_workload(args):
    from paper_2401_06104_b200 import workloads as W
    w = W.WORKLOADS[args.workload]
    if args.capacity:
        w = w.scaled(capacity=args.capacity)
    if args.batch:
        w = w.scaled(batch=args.batch)
    return w


# ----------------------------------------------------------------------------
# clocks: sampled with NVML (read-only) while the timed region runs
# ----------------------------------------------------------------------------
class ClockSampler:
    BAD = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown"}
    NOTE = {0x4: "sw_power_cap"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            if vis:
                index = int(vis.split(",")[index]) if vis.split(",")[index].isdigit() else index
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                for bit, name in {**self.BAD, **self.NOTE}.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.005)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ----------------------------------------------------------------------------
# the CPU checker as a timed baseline (never tuned for this)
# ----------------------------------------------------------------------------
def time_oracle(w, ring, seconds: float, max_seqs: int = 0):
    """Steady-state decode steps of the CPU checker on a full state.  The state
    is written directly from ring tokens (while filling nothing is dropped), then
    steps are timed.  Returns (tokens/s, threads, description)."""
    from oracle.tova_oracle import OracleCache, host_threads
    threads = host_threads()
    S = min(w.batch, max_seqs or max(threads, 1))
    q, k, v = ring
    orc = OracleCache(S, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, precision="f32", threads=threads)
    R = q.shape[0]
    for n in range(w.capacity):
        orc.K[:, :, n] = k[n % R][:S]
        orc.V[:, :, n] = v[n % R][:S]
        orc.pos[:, n] = n
    orc.len[:] = w.capacity
    pos = w.capacity
    t0 = time.perf_counter()
    orc.step(q[0][:S], k[0][:S], v[0][:S], pos); pos += 1
    one = max(time.perf_counter() - t0, 1e-6)
    n_steps = int(min(max(seconds / one, 4), 4096))
    t0 = time.perf_counter()
    for i in range(n_steps):
        r = (i + 1) % R
        orc.step(q[r][:S], k[r][:S], v[r][:S], pos); pos += 1
    dt = time.perf_counter() - t0
    used = min(threads, S)
    return S * n_steps / dt, used, f"{n_steps} steady-state steps of {S} of {w.batch} sequences on a full state (k={w.capacity})"


def storage_name(w):
    """Type of q, k, v and the cached rows; sums and soft-max run in fp32."""
    return "bf16" if w.elem_bytes == 2 else "f32"


def workload_config(w, extra):
    cfg = {"workload": w.name, "batch": w.batch, "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads,
           "head_dim": w.head_dim, "capacity": w.capacity,
           "storage": "bf16" if w.elem_bytes == 2 else "fp32"}
    cfg.update(extra)
    return cfg


def run_reference(args):
    """--impl reference: the CPU checker alone, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_2401_06104_b200 import workloads as W
    w = pick_workload(args)
    ring = W.tokens(w, 0, RING)
    # every "step" is a bounded sample; the whole run stays within minutes
    seconds = min(60.0, max(4.0, 0.004 * (args.steps + args.warmup)))
    val, cores, sample = time_oracle(w, ring, seconds)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * w.batch / val,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": workload_config(w, {"l2": "not applicable: host cores", "parallelism": "replicas only" if args.gpus > 1 else "single GPU"}),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------
# the CUDA path
# ----------------------------------------------------------------------------
# Sources of the streaming (split) kernels, the ones the recorded DRAM counters describe.
SPLIT_KERNEL_SOURCES = ("tova_device.cuh", "tova_kernels.cuh", "tova_split_mma.cuh")


def kernel_digest() -> str:
    """Hash of the streaming kernels' sources: DRAM counters in profiles/ apply to one digest only."""
    import hashlib
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2401_06104_b200", "csrc")
    for f in SPLIT_KERNEL_SOURCES:
        with open(os.path.join(d, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def recorded_traffic(w, layers_bytes_per_step):
    """DRAM bytes per split-kernel launch from the committed ncu summary, or None
    when there is none for this workload or the kernels changed since."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        with open(path) as fh:
            rec = json.load(fh)
        if rec.get("kernel_digest") != kernel_digest():
            return None
        e = rec["workloads"].get(f"{w.name}:k{w.capacity}:b{w.batch}")
        return None if e is None else float(e["dram_bytes_per_launch"])
    except Exception:
        return None


def max_over_ranks(x: float, device) -> float:
    """Max of a host number over all ranks (1 rank: the number itself)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


MIN_TIMED_MS = 50.0             # the K timed steps are repeated until the timed region lasts at least this long

# The other roofline-graded configurations (state of 1024 rows and more), timed after the headline in the same
# run: (workload, capacity, layer caches).
SWEEP = [("mistral_7b_gqa", 1024, 0), ("mistral_7b_gqa", 4096, 0), ("yi_6b_long", 4096, 0),
         ("llama2_7b_full", 8192, 2)]


def measure(w, args, dev, world, layers=0, want_e2e=False):
    """Steady-state decode steps of workload `w` on the current device: fills `layers` caches past their capacity,
    captures args.steps steps as one CUDA graph and replays it until the timed region lasts MIN_TIMED_MS.
    Returns a dict of measurements (host numbers; times are the max over ranks)."""
    import torch
    import torch.distributed as dist

    import paper_2401_06104_b200 as tova
    from paper_2401_06104_b200 import workloads as W

    B, H, Hkv, D, cap = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity
    step_bytes = w.step_bytes()
    # at least two layers: consecutive steps then belong to different caches, as in a model
    L = layers or args.layers or min(64, max(2, w.n_layers, -(-WORKING_SET // step_bytes)))
    deferred = (not args.no_deferred and L >= 2) or args.deferred
    ring = W.tokens(w, 0, RING)                                   # seeded, host
    dq, dk, dv = (tova.to_device(a, w.dtype, dev) for a in ring)

    caches = []
    for l in range(L):
        c = tova.TovaCache(B, H, Hkv, D, cap, dtype=w.dtype, device=dev)
        if args.chunk_rows:
            c.tova_cache_set_chunk_rows(args.chunk_rows)
        if args.no_fused_merge:
            c.tova_cache_set_fused_merge(False)
        if args.position_compression:
            c.tova_cache_set_position_compression(args.position_compression)
        if args.policy != "tova" or args.keep_first:
            c.tova_cache_set_policy({"tova": tova.TOVA_POLICY_TOVA, "window": tova.TOVA_POLICY_WINDOW,
                                     "tova_head": tova.TOVA_POLICY_TOVA_HEAD, "h2o_layer": tova.TOVA_POLICY_H2O_LAYER,
                                     "h2o_head": tova.TOVA_POLICY_H2O_HEAD}[args.policy], args.keep_first)
        caches.append(c)
    outs = torch.empty(L, B, H, D, dtype=torch.float32, device=dev)
    evs = torch.empty(L, B, caches[0].tova_cache_units(), dtype=torch.int32, device=dev)

    # steady state: fill every layer past its capacity (positions from the device counter)
    for l, c in enumerate(caches):
        fed, r = 0, (17 * l) % RING
        while fed < cap + 16:
            T = min(RING - r, cap + 16 - fed)
            c.tova_prefill(dq[r:], dk[r:], dv[r:], T, -1, None, None)
            fed += T
            r = (r + T) % RING
    torch.cuda.synchronize()
    for c in caches:
        assert c.tova_cache_len() == cap
        if deferred:
            c.tova_cache_set_deferred_eviction(True)

    def join_all():
        if deferred:
            for c in caches:
                c.tova_cache_join()

    counter = [0]

    def step(i):
        l = i % L
        r = (i // L + 29 * l) % RING
        caches[l].tova_decode_step(dq[r], dk[r], dv[r], -1, outs[l], evs[l])

    def run_direct(n):
        for _ in range(n):
            step(counter[0])
            counter[0] += 1

    # Warm-up, part 1: host-launched steps, at least one per cache (sets function attributes before capture).
    l0 = sum(c.tova_cache_launches() for c in caches)
    n_direct = max(args.warmup, 3, L)
    run_direct(n_direct)
    launches_per_step = (sum(c.tova_cache_launches() for c in caches) - l0) / n_direct
    join_all()
    torch.cuda.synchronize()

    # The K timed steps as ONE graph of C-ABI calls, whatever K is.
    K = args.steps
    graph = None
    launch_mode = "stream"
    if not args.no_graph:
        try:
            graph = torch.cuda.CUDAGraph()
            base = counter[0]
            with torch.cuda.graph(graph):
                for j in range(K):
                    step(base + j)
                join_all()                                        # side streams rejoin before the capture ends
            launch_mode = "cuda_graph"
        except Exception as e:  # pragma: no cover
            print(f"bench.py: graph capture failed ({e}); launching from the host", file=sys.stderr)
            graph = None
            torch.cuda.synchronize()

    def run_k():
        if graph is not None:
            graph.replay()
        else:
            run_direct(K)
            join_all()

    # Warm-up, part 2: the timed unit itself, and an estimate of how often to repeat it.
    for _ in range(2):
        run_k()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    run_k()
    e1.record()
    torch.cuda.synchronize()
    est = max(max_over_ranks(e0.elapsed_time(e1), dev), 1e-3)
    repeats = args.repeats or max(1, int(-(-MIN_TIMED_MS // est)) + 1)

    sampler = ClockSampler(torch.cuda.current_device())
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    e0.record()
    for _ in range(repeats):
        run_k()
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if world > 1:
        dist.barrier()
    ms = max_over_ranks(e0.elapsed_time(e1), dev)
    for c in caches:
        assert c.tova_cache_read()["status"] == 0, "a kernel reported a failed check"

    timed_steps = repeats * K
    ms_per_step = ms / timed_steps
    res = {
        "ms": ms, "ms_per_step": ms_per_step, "timed_steps": timed_steps, "repeats": repeats,
        "value": world * B * timed_steps / (ms * 1e-3), "gbs": step_bytes / (ms_per_step * 1e-3) / 1e9,
        "launch": launch_mode, "layers": L, "deferred": deferred, "step_bytes": step_bytes,
        "launches": int(round(launches_per_step * timed_steps)), "clocks": clocks, "ring": ring, "e2e": None,
    }

    # end to end: host buffers in, host buffers out, through tova_decode_step_host
    if want_e2e:
        hq, hk, hv = (torch.from_numpy(a).to(dq.dtype).pin_memory() for a in ring)
        hout = torch.empty(B, H, D, dtype=torch.float32).pin_memory()
        hev = torch.empty(B, evs.shape[2], dtype=torch.int32).pin_memory()
        n_e = max(K, min(2048, int(4 * MIN_TIMED_MS / ms_per_step) + 1))
        for i in range(max(8, L)):
            caches[i % L].tova_decode_step_host(hq[i % RING], hk[i % RING], hv[i % RING], -1, hout, hev)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for i in range(n_e):
            r = (i // L + 29 * (i % L)) % RING
            caches[i % L].tova_decode_step_host(hq[r], hk[r], hv[r], -1, hout, hev)
        torch.cuda.synchronize()
        dt = max_over_ranks(time.perf_counter() - t0, dev)
        res["e2e"] = {"value": world * B * n_e / dt, "unit": UNIT, "steps": n_e,
                      "h2d_bytes_per_step": int(hq[0].nbytes + hk[0].nbytes + hv[0].nbytes),
                      "d2h_bytes_per_step": int(hout.nbytes + hev.nbytes)}
    for c in caches:
        c.close()
    del caches, outs, evs, graph
    torch.cuda.empty_cache()
    return res


def roofline_of(w, res, peak, peak_kind):
    return {"bound": "hbm", "achieved": res["gbs"], "peak": peak, "unit": "GB/s", "frac": res["gbs"] / peak,
            "traffic": recorded_traffic(w, res["step_bytes"]), "peak_kind": peak_kind,
            "frac_of_nominal_8TBs": res["gbs"] / 8000.0,
            "note": "algorithmic bytes (K/V read + one slot written) / whole-step time (split + combine kernels)"}


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2401_06104_b200 import workloads as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the decode path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    w = pick_workload(args)
    peak, peak_kind = load_peaks()
    res = measure(w, args, dev, world, want_e2e=not args.no_e2e)
    L, step_bytes = res["layers"], res["step_bytes"]

    # the other graded configurations, one GPU only (with several ranks all of them would be held meanwhile)
    sweep = []
    if world == 1 and not args.no_sweep and args.workload == DEFAULT_WORKLOAD and not args.capacity and not args.batch:
        for name, capacity, layers in SWEEP:
            ws = W.WORKLOADS[name].scaled(capacity=capacity)
            r = measure(ws, args, dev, world, layers=layers)
            sweep.append({"workload": name, "capacity": capacity, "batch": ws.batch, "bytes_per_step": r["step_bytes"],
                          "layers_rotated": r["layers"], "ms_per_step": r["ms_per_step"], "value": r["value"],
                          "achieved_gbs": r["gbs"], "frac": r["gbs"] / peak, "launch": r["launch"],
                          "timed_steps": r["timed_steps"], "timed_ms": r["ms"], "clocks": r["clocks"]})

    if rank != 0:
        return 0

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        val, cores, sample = time_oracle(w, res["ring"], args.cpu_seconds)
        cpu = {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}

    line = {
        "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": res["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": storage_name(w), "data": "synthetic",
        "timed_steps": res["timed_steps"], "repeats": res["repeats"], "timed_ms": res["ms"],
        "config": workload_config(w, {
            "l2": "inputs larger than L2" if min(L, args.steps) * step_bytes > 2 * 126e6
                  else "working set near or below L2 size",
            "parallelism": "replicas only" if world > 1 else "single GPU"}),
        "run": {
            "layers_rotated": L, "working_set_bytes": min(L, args.steps) * step_bytes,
            "launch": res["launch"], "graph_steps": args.steps if res["launch"] == "cuda_graph" else 0,
            "bytes_per_step": step_bytes, "accumulate": "fp32",
            "policy": args.policy + (f"+{args.keep_first}" if args.keep_first else ""),
            "eviction": "deferred to the cache's side stream, overlaps the next layer's step" if res["deferred"]
                        else "on the caller's stream"},
        "roofline": roofline_of(w, res, peak, peak_kind),
        "cpu_baseline": cpu,
        "e2e": res["e2e"],
        "gpu_launches": res["launches"],
        "clocks": res["clocks"],
        "sweep": sweep,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def run_prefill(args):
    """Prompt processing: one tova_prefill call of T tokens into an empty state per step (a fresh cache each
    step, so inputs and state are cold).  One GPU.  Roofline of the bulk route: the causal-attention kernel,
    2*B*H*D*F*(F+1) flops for the F tokens that find a free row, against the measured bf16 GEMM rate."""
    import torch
    import paper_2401_06104_b200 as tova
    from paper_2401_06104_b200 import workloads as W
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the prefill path has no CPU fallback")
    dev = "cuda:0"
    torch.cuda.set_device(0)
    w = pick_workload(args)
    B, H, Hkv, D, cap = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity
    T = cap if args.prefill < 0 else args.prefill
    steps, warm = min(args.steps, 8), min(max(args.warmup, 3), 3)
    q, k, v = (tova.to_device(a, w.dtype, dev) for a in W.tokens(w, 0, T))
    out = torch.empty(T, B, H, D, dtype=torch.float32, device=dev)
    caches = []
    chunked = not (args.no_chunked_prefill or args.no_bulk_prefill) and w.dtype == W.DTYPE_BF16 and T > cap
    ws = None
    for _ in range(steps + warm):
        c = tova.TovaCache(B, H, Hkv, D, cap, dtype=w.dtype, device=dev)
        if args.no_bulk_prefill or args.warp_mma_prefill:
            c.tova_cache_set_bulk_prefill(0 if args.no_bulk_prefill else 2)
        if args.policy != "tova" or args.keep_first:
            c.tova_cache_set_policy({"tova": tova.TOVA_POLICY_TOVA, "window": tova.TOVA_POLICY_WINDOW,
                                     "tova_head": tova.TOVA_POLICY_TOVA_HEAD, "h2o_layer": tova.TOVA_POLICY_H2O_LAYER,
                                     "h2o_head": tova.TOVA_POLICY_H2O_HEAD}[args.policy], args.keep_first)
        if chunked:
            ws = c.tova_cache_set_prefill_workspace(ws)          # one workspace serves all: calls share a stream
            if args.chunk_cluster:
                c.tova_cache_set_chunk_cluster(args.chunk_cluster)
            if args.chunk_barriers:
                c.tova_cache_set_chunk_barriers(args.chunk_barriers)
        caches.append(c)
    ev = torch.empty(T, B, caches[0].tova_cache_units(), dtype=torch.int32, device=dev)   # per unit for head-wise policies
    torch.cuda.synchronize()
    for c in caches[:warm]:
        c.tova_prefill(q, k, v, T, 0, out, ev)
    sampler = ClockSampler(0)
    torch.cuda.synchronize()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for c in caches[warm:]:
        c.tova_prefill(q, k, v, T, 0, out, ev)
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    for c in caches:
        assert c.tova_cache_read()["status"] == 0, "a kernel reported a failed check"
    ms = e0.elapsed_time(e1) / steps
    launches = caches[-1].tova_cache_launches() - 1
    F = min(T, cap)
    flops = 2.0 * B * H * D * F * (F + 1)
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            peak, kind = float(json.load(fh)["bf16_tflops"]), "measured"
    except Exception:
        peak, kind = 1590.0, "fallback"
    bulk = (not args.no_bulk_prefill) and w.dtype == W.DTYPE_BF16 and F >= 4
    line = {
        "metric": "tova_prefill_tokens_per_s_per_layer", "value": B * T / (ms * 1e-3), "unit": UNIT, "n_gpus": 1,
        "steps": steps, "warmup": warm, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": storage_name(w), "data": "synthetic",
        "config": workload_config(w, {"prompt_tokens": T, "tokens_into_free_rows": F,
                                      "route": ("bulk fill + chunks of 64" if chunked else "bulk fill + per-token steps") if bulk
                                               else "per-token steps",
                                      "l2": "a fresh cache per step; inputs larger than L2" if q.numel() * 2 > 126e6
                                            else "a fresh cache per step",
                                      "parallelism": "single GPU"}),
        "roofline": ({"bound": "tensor", "achieved": flops / (ms * 1e-3) / 1e12, "peak": peak, "unit": "TFLOP/s",
                      "frac": flops / (ms * 1e-3) / 1e12 / peak, "traffic": None, "peak_kind": kind,
                      "note": "causal-attention flops of the bulk run / whole prefill time; "
                              + ("warp-level MMA kernel" if args.warp_mma_prefill or D != 128 else "tcgen05 kernel")}
                     if bulk and T == F else None),
        "cpu_baseline": None, "e2e": None, "gpu_launches": launches * steps, "clocks": clocks,
    }
    print(json.dumps(line))
    return 0


def main():
    args = parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.prefill:
        return run_prefill(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
