#!/usr/bin/env python
"""Benchmark of the LESS decode hot path on B200.

A step = one generation step (Algorithm 1) of every (batch, layer, head)
instance of the workload: feature maps, attention over the kept slots with the
low-rank correction, score update, eviction, state update.  The cache is first
built by the library's own prompt phase from seeded synthetic Q/K/V, then
`--warmup` untimed steps run, then blocks of exactly `--steps` steps are timed
(CUDA events, a barrier + synchronize on both sides of every block) until there
are at least 20 blocks and 0.5 s of device time; the line reports the median
block (and the fastest).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

Without --config the line's headline is the batched-serving workload (cfg3, the
largest that decodes on one GPU) and the other four workloads ride along as
sub-records under "configs" (cfg5 = prompt compression, one layer per step).
Prints ONE JSON line (rank 0).  With --impl reference the fp64 CPU oracle is
timed instead, on a bounded sample of the same workload.  With --gpus N > 1 and
no torchrun environment the script starts its own N ranks (one replica per GPU).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode attention head-tokens/s (B x layers x heads per step)"
UNIT = "head-tokens/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_TFLOPS = 1400.0
NOMINAL_HBM_GBS = 8000.0
MIN_BLOCKS, MIN_DEVICE_MS = 20, 500.0
HEADLINE_CONFIG = 3


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20, help="steps per timed block")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=0,
                    help="workload id (1-4 decode; 5 = prompt compression, one layer per step; 6 = the multi-query "
                         "shape of Section 4, context run); "
                         "0 = cfg3 as the headline plus sub-records for the other four")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="budget of the CPU-baseline leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--blocks", type=int, default=0,
                    help="time exactly this many blocks (default: at least 20 and 0.5 s of device time); "
                         "small values keep profiler captures short")
    ap.add_argument("--full-cache", action="store_true",
                    help="context run: slots >= prompt + steps, so nothing is ever evicted")
    ap.add_argument("--no-state", action="store_true", help="context run: sparse policy alone (Baseline+)")
    ap.add_argument("--lambda-masking", action="store_true",
                    help="context run: Lambda-masking as the sparse policy (first 4 tokens + window, same slot count)")
    ap.add_argument("--graph", action="store_true",
                    help="launch the decode steps as replays of a CUDA graph of 8 captured steps "
                         "(for launch-bound workloads such as cfg1)")
    ap.add_argument("--tova", action="store_true",
                    help="context run: TOVA as the sparse policy (same slot count)")
    ap.add_argument("--attn-out", action="store_true",
                    help="prompt compression: also produce the prompt's attention output (optional in less_prefill)")
    ap.add_argument("--masked-form", action="store_true",
                    help="context run: the parallel form (training / evaluation): sequences of --seq tokens, batch 2, "
                         "32 heads, one layer per step")
    ap.add_argument("--seq", type=int, default=4096, help="sequence length of --masked-form")
    ap.add_argument("--group", type=int, default=1, choices=[1, 2, 4, 8],
                    help="context run: grouped query heads, G query heads per KV head (query heads unchanged, "
                         "KV heads divided by G)")
    ap.add_argument("--batch", type=int, default=0,
                    help="override the workload's batch (smaller captures for ncu; named in config.workload)")
    ap.add_argument("--out-f16", action="store_true", help="fp16 attention output (LESS_OUT_F16)")
    return ap.parse_args(argv)


def peaks():
    """(HBM GB/s, sustained 16-bit TFLOP/s, 'measured' | 'fallback')."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d["bf16_tflops_sustained"]), "measured"
    return FALLBACK_HBM_GBS, FALLBACK_TFLOPS, "fallback"


# --------------------------------------------------------------------------- #
# algorithmic bytes per launch
# --------------------------------------------------------------------------- #
def feature_map_bytes(w, no_state=False):
    if no_state:
        return 0
    D, Rp, R, G = w.head_dim, w.hidden, w.rank, w.group
    weights = w.layers * w.heads * ((G + 1) * (D * Rp + Rp * R) + R * R) * 2    # phi per query head, psi per KV head
    io = w.instances * ((G + 1) * D * 2 + (G + 1) * R * 4)
    return weights + io


def decode_bytes(w, n_live, evicting=True, no_state=False, out_bytes=4):
    D, R, G = w.head_dim, w.rank, w.group
    per = n_live * (2 * D * 2)              # K and V rows
    per += n_live * (4 + 4)                 # accumulated score read + write
    per += n_live * 4 if evicting else 0    # positions (only read when a victim is needed)
    per += (2 + G) * D * 2 + G * D * out_bytes   # q, k, v in; out (G query heads per KV head)
    per += 2 * D * 2 + 8                    # new pair into its slot, pos, acc
    per += 4                                # slot count
    if not no_state:
        per += R * D * 4 + R * 4            # H, z read
        per += (G + 1) * R * 4              # phi(q) of the G heads, psi(k) read
        per += R * 4                        # psi into the slot's cache
        if evicting:
            per += R * D * 4 + R * 4 + R * 4 + D * 2   # H, z write; victim psi; victim v row
    return w.instances * per


def kv_state_scores_bytes(w, n_live, no_state=False):
    """Bytes of the kept K / V rows, the low-rank state (read and written) and the accumulated
    scores (read and written) of one step: the narrow roofline that leaves the feature-map
    weights, positions and the step's inputs and outputs out."""
    return w.instances * (n_live * (4 * w.head_dim + 8) + (0 if no_state else 2 * w.rank * w.head_dim * 4))


# --------------------------------------------------------------------------- #
# measured DRAM traffic per launch (profiles/traffic.json: data only)
# --------------------------------------------------------------------------- #
def _sha16(path):
    try:
        return hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]
    except OSError:
        return None


def ncu_traffic(workload_key, kernel_key):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of `kernel_key` on `workload_key`
    from the tracked capture table, or None: no capture, or the kernel's source file has changed
    since the counters were taken (the table stores the file's hash at capture time)."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(path):
        return None, "no capture table"
    for e in json.load(open(path))["captures"]:
        if e["workload"] == workload_key and e["kernel_key"] == kernel_key:
            now = _sha16(os.path.join(ROOT, e["source"]))
            if now != e["source_sha256_16"]:
                return None, f"capture of {e['captured']} is stale: {e['source']} changed since"
            return float(e["bytes_per_launch"]), e.get("note", f"captured {e['captured']}")
    return None, "no capture of this kernel and workload"


# --------------------------------------------------------------------------- #
# ranks: replicas only; what the ranks exchange is the timing
# --------------------------------------------------------------------------- #
def max_over_ranks(values, device, world):
    """Replicas only: every rank runs the whole workload on its own GPU and the job's time is the
    slowest rank's.  Element-wise maximum of `values` over the ranks (identity for one rank)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def job_throughput(units_per_rank, steps, ms, world):
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    return units_per_rank * world * steps / (ms * 1e-3)


def timed_blocks(time_block, reduce_max, min_blocks=MIN_BLOCKS, min_total_ms=MIN_DEVICE_MS, exact_blocks=0,
                 max_blocks=5000, max_wall_s=30.0):
    """Times blocks until there are `min_blocks` of them and `min_total_ms` of timed duration
    (or exactly `exact_blocks`).  `time_block()` runs and times one block on this rank (ms);
    `reduce_max([ms])` turns it into the slowest rank's, so every rank sees the same durations
    and stops after the same block.  Returns the list of block durations."""
    times, wall0 = [], time.time()
    while True:
        times.append(reduce_max([time_block()])[0])
        n, total = len(times), sum(times)
        if exact_blocks:
            if n >= exact_blocks:
                break
            continue
        over = reduce_max([1.0 if time.time() - wall0 > max_wall_s else 0.0])[0] > 0
        if (n >= min_blocks and total >= min_total_ms) or n >= max_blocks or (over and n >= min_blocks):
            break
    return times


def block_stats(times, steps):
    return {"ms_per_step": statistics.median(times) / steps, "ms_per_step_min": min(times) / steps,
            "blocks": len(times), "timed_device_ms": sum(times)}


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_ranks(n, script, argv, require_gpus=True, timeout=None):
    """Starts `script argv` as n ranks of one node (one process per GPU, rendezvous on
    127.0.0.1) and returns the launcher's exit code.  With require_gpus the node must have n
    CUDA devices: fewer is an error, never a silent run on fewer."""
    if require_gpus:
        import torch
        have = torch.cuda.device_count() if torch.cuda.is_available() else 0
        if have < n:
            raise SystemExit(f"bench.py --gpus {n}: this node has {have} CUDA device(s); "
                             f"refusing to run {n} ranks on fewer GPUs")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), script] + list(argv)
    return subprocess.call(cmd, timeout=timeout)


class Ranks:
    """This process's place among the ranks, its device, and the barrier of the timed regions."""

    def __init__(self):
        import torch
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        if not torch.cuda.is_available():
            raise RuntimeError("bench.py needs a CUDA device: the LESS path has no CPU fallback")
        torch.cuda.set_device(self.local)
        self.dev = f"cuda:{self.local}"
        if self.world > 1:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=torch.device(self.dev))

    def barrier(self):
        import torch
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    def reduce_max(self, values):
        return max_over_ranks(values, self.dev, self.world)

    def close(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


def cuda_block_timer(ranks, stream, run_block):
    """time_block() for timed_blocks: barrier + synchronize, event, the block, event, barrier +
    synchronize; the events are recorded on the stream the kernels are launched on."""
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def time_block():
        ranks.barrier()
        e0.record(stream)
        run_block()
        e1.record(stream)
        ranks.barrier()
        return e0.elapsed_time(e1)
    return time_block


class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML (read-only) every
    5 ms on a thread while the timed region runs."""

    def __init__(self, index):
        self.samples, self.stop_flag, self.ok = [], False, False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            # honour CUDA_VISIBLE_DEVICES when it lists indices
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            phys = index
            if vis and all(x.strip().isdigit() for x in vis.split(",")):
                phys = int(vis.split(",")[index])
            self.h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception as e:  # no NVML: report that, never guess
            self.err = repr(e)

    def _pump(self):
        nv = self.nv
        while not self.stop_flag:
            try:
                mhz = float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                rs = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                self.samples.append((time.time(), mhz, rs))
            except Exception:
                pass
            time.sleep(0.005)

    def stop(self, t0, t1):
        if not self.ok:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["NVML unavailable: " + getattr(self, "err", "")]}
        self.stop_flag = True
        self.thread.join(timeout=1.0)
        nv = self.nv
        rows = [(m, r) for (t, m, r) in self.samples if t0 <= t <= t1] or [(m, r) for _, m, r in self.samples]
        sm = sorted(m for m, _ in rows)
        names = {"hw_slowdown": nv.nvmlClocksEventReasonHwSlowdown,
                 "hw_thermal_slowdown": nv.nvmlClocksEventReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": nv.nvmlClocksEventReasonSwThermalSlowdown,
                 "sw_power_cap": nv.nvmlClocksEventReasonSwPowerCap,
                 "hw_power_brake": nv.nvmlClocksEventReasonHwPowerBrakeSlowdown}
        reasons = sorted(n for n, bit in names.items() if any(r & bit for _, r in rows))
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_min_mhz": sm[0] if sm else None,
                "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(sm)}


# --------------------------------------------------------------------------- #
# CPU oracle timing (cpu_baseline leg and --impl reference)
# --------------------------------------------------------------------------- #
def _oracle_worker(job):
    """One worker process of the CPU baseline (no torch, no CUDA in here): builds its share of the
    sampled instances from their records and times oracle decode steps, one numpy thread."""
    from threadpoolctl import threadpool_limits
    from oracle import less_oracle as lo
    D, R, heavy, recent, weights, records, q, k, v, seconds = job
    with threadpool_limits(limits=1):
        orcs = []
        for wts, r in zip(weights, records):
            o = lo.LessInstance(D, R, heavy, recent, *lo.make_mlp_maps(*wts))
            o.import_state(r["pos"], r["K"], r["V"], r["acc"], r["H"], r["z"], r["t"])
            orcs.append(o)
        units, steps, t0 = 0, 0, time.perf_counter()
        while True:                                   # the step inputs are used round-robin until the time is up
            s = steps % q.shape[0]
            for i, o in enumerate(orcs):
                o.decode(q[s, i], k[s, i], v[s, i])
            units += len(orcs)
            steps += 1
            if time.perf_counter() - t0 > seconds or steps >= 100000:
                break
        return units, time.perf_counter() - t0, steps


def oracle_rate(w, seconds, records=None, instances=None, W=None, max_instances=16, max_steps=64):
    """Times oracle decode steps on a bounded sample of instances (`seconds` of CPU work in total), the
    instances spread over worker processes on the host's cores (the oracle itself is untouched: one numpy
    thread per instance; the sampled steps' inputs are reused round-robin until the time is up).  With
    `records` (states exported from the GPU) the oracle starts from them, else it runs its own prompt
    phase first (untimed).  Returns (head-tokens/s, cores, text, steps, s)."""
    import multiprocessing as mp
    from concurrent.futures import ProcessPoolExecutor
    import numpy as np
    from oracle import less_oracle as lo
    from paper_2402_09398_b200 import workloads as wl
    if W is None:
        W = wl.make_weights(w, "cpu")
    if instances is None:
        instances = list(range(0, w.instances, max(1, w.instances // max_instances)))[:max_instances]
    weights, prompt_cache = [], {}
    built = records is None
    if built:
        records = []
    for n, inst in enumerate(instances):
        b, layer, head = wl.instance_coords(w, inst)
        wts = [W[k][layer, head].double().cpu().numpy() for k in ("w_phi1", "w_phi2", "w_psi1", "w_psi2", "w_psi3")]
        weights.append(wts)
        if built:
            if layer not in prompt_cache:
                prompt_cache = {layer: wl.make_prompt(w, layer, 1, "cpu")}
            Q, K, V = prompt_cache[layer]
            o = lo.LessInstance(w.head_dim, w.rank, w.heavy, w.recent, *lo.make_mlp_maps(*wts))
            o.prefill(*(t[b, 0, head].double().numpy() for t in (Q, K, V)))
            records.append({"pos": o.pos, "K": o.K, "V": o.V, "acc": o.acc, "H": o.H, "z": o.z, "t": o.t})
    # decode inputs of the sampled instances only (the generators draw whole steps)
    nsteps = max(1, min(max_steps, w.steps if w.steps else max_steps))
    idx = np.asarray(instances)
    qs, ks, vs = [], [], []
    for s in range(nsteps):
        q, k, v = wl.make_decode_inputs(w, s, "cpu")
        qs.append(q.reshape(-1, w.head_dim)[idx].double().numpy())
        ks.append(k.reshape(-1, w.head_dim)[idx].double().numpy())
        vs.append(v.reshape(-1, w.head_dim)[idx].double().numpy())
    q, k, v = np.stack(qs), np.stack(ks), np.stack(vs)               # [steps, instances, D]
    try:
        avail = len(os.sched_getaffinity(0))
    except AttributeError:
        avail = os.cpu_count() or 1
    cores = max(1, min(avail, len(instances), 16))
    shares = [list(range(c, len(instances), cores)) for c in range(cores)]
    # `seconds` = CPU work in total: every worker runs for its share of it
    jobs = [(w.head_dim, w.rank, w.heavy, w.recent, [weights[i] for i in sh], [records[i] for i in sh],
             q[:, sh], k[:, sh], v[:, sh], seconds / cores) for sh in shares]
    if cores == 1:
        results = [_oracle_worker(jobs[0])]
    else:
        with ProcessPoolExecutor(max_workers=cores, mp_context=mp.get_context("spawn")) as pool:
            results = list(pool.map(_oracle_worker, jobs))
    units = sum(r[0] for r in results)
    t_used = max(r[1] for r in results)
    steps = max(r[2] for r in results)
    sample = (f"{len(instances)} of {w.instances} instances x {steps} decode steps "
              f"({'oracle-prefilled' if built else 'GPU-exported'} state), fp64 numpy, one thread per instance, "
              f"{cores} worker process(es) on {avail} available core(s)")
    return units / t_used, cores, sample, steps, t_used


def oracle_prompt_rate(w, prompt, seconds):
    """Times the oracle's prompt phase (scoring, selection, state build) of single heads whose
    prompt is cut to `prompt` tokens: the full length is hours of fp64 work per head."""
    from threadpoolctl import threadpool_limits
    from oracle import less_oracle as lo
    from paper_2402_09398_b200 import workloads as wl
    ws = w.with_(batch=1, layers=1, heads=2, prompt=prompt, heavy=int(0.05 * prompt), recent=int(0.05 * prompt))
    W = wl.make_weights(ws, "cpu")
    Q, K, V = wl.make_prompt(ws, 0, 1, "cpu")
    tokens, t_used, n = 0, 0.0, 0
    with threadpool_limits(limits=1):
        while t_used < seconds and n < ws.heads:
            wts = [W[k][0, n].double().numpy() for k in ("w_phi1", "w_phi2", "w_psi1", "w_psi2", "w_psi3")]
            o = lo.LessInstance(ws.head_dim, ws.rank, ws.heavy, ws.recent, *lo.make_mlp_maps(*wts))
            t0 = time.perf_counter()
            o.prefill(*(t[0, 0, n].double().numpy() for t in (Q, K, V)))
            t_used += time.perf_counter() - t0
            tokens += prompt
            n += 1
    sample = (f"{n} head(s), prompt cut to {prompt} of {w.prompt} tokens (the scoring cost grows with the square "
              f"of the length, so the full-length rate is lower), fp64 numpy, 1 thread")
    return tokens / t_used, 1, sample


def run_reference(args):
    from paper_2402_09398_b200 import workloads as wl
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = args.config or HEADLINE_CONFIG
    w = wl.CONFIGS[cfg]
    if cfg == 5:
        rate, cores, sample = oracle_prompt_rate(w, 2048, 60.0)
        line = {"impl": "reference", "metric": PROMPT_METRIC, "value": rate, "unit": UNIT, "n_gpus": 0,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": None, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "config": {"workload": workload_name(w, args)},
                "cpu_baseline": {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
                "e2e": {"value": rate, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return
    # each "step" = one oracle decode step over a bounded sample of instances (8 heads of the first
    # batch rows: the per-instance work does not depend on the batch)
    n_inst = 8
    w_run = w.with_(batch=min(w.batch, 2), steps=args.steps + args.warmup)
    rate, cores, sample, steps_done, t_used = oracle_rate(w_run, seconds=60.0, max_instances=n_inst)
    sample = sample.replace(f"of {w_run.instances} instances", f"of {w.instances} instances")
    line = {
        "impl": "reference", "metric": METRIC, "value": rate, "unit": UNIT, "n_gpus": 0,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_used / max(1, steps_done),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(w, args),
        "cpu_baseline": {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": rate, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


WORKLOAD_NAMES = {
    1: "cfg1 smallest (B=1, 1 layer x 8 heads, prompt 256, 32+32 slots, R=8)",
    2: "cfg2 Llama-2-7B shape (B=1, 32 layers x 32 heads, prompt 2048, 102+102 slots, R=8)",
    3: "cfg3 batched serving (B=64, 32 layers x 32 heads, prompt 1024, 102+102 slots, R=8)",
    4: "cfg4 long context (B=4, 40 layers x 40 heads, prompt 16384, 327+327 slots, R=16)",
    5: "cfg5 prefill compression (B=8, 32 heads, one layer per step, prompt 32768, 1638+1638 slots, R=16)",
    6: "multi-query shape (B=64, 32 layers x 1 KV head x 71 query heads, D=64, 102+102 slots filled by decoding, R=8)",
}
PROMPT_METRIC = "prompt head-tokens/s (prompt scoring, selection, state build; one layer per step)"


def workload_name(w, args):
    name = WORKLOAD_NAMES[w.cfg_id]
    if getattr(args, "batch", 0):
        name += f" [batch set to {w.batch} for profiling]"
    return name


def workload_config(w, args):
    c = {"workload": workload_name(w, args), "instances": w.instances, "slots": w.slots, "rank": w.rank,
         "prompt": w.prompt, "l2": "bytes touched per step exceed the 126 MB L2"
         if w.cfg_id != 1 else "L2 flushed by a 256 MB write between steps is NOT done: cfg1 is launch-bound"}
    if getattr(args, "full_cache", False):
        c["variant"] = "full cache (no eviction)"
    if getattr(args, "graph", False):
        c["launch"] = "replays of a CUDA graph of 8 captured steps"
    if getattr(args, "tova", False):
        c["variant"] = "TOVA policy (lowest probability of the current query leaves)"
    if getattr(args, "lambda_masking", False):
        c["variant"] = "Lambda-masking policy (first 4 tokens + recent window)"
    if getattr(args, "no_state", False):
        c["variant"] = "sparse policy alone (Baseline+)"
    if getattr(args, "group", 1) > 1:
        c["variant"] = (f"grouped query heads: {w.heads} KV heads x {w.group} query heads per layer; "
                        "the unit counts query heads")
    if getattr(args, "out_f16", False):
        c["output"] = "fp16"
    return c


# --------------------------------------------------------------------------- #
# decode workloads (cfg1 - cfg4)
# --------------------------------------------------------------------------- #
def measure_decode(args, ranks, cfg_id, cpu_seconds):
    """Builds the cache of workload `cfg_id` with the library's prompt phase, then times decode
    steps three ways (device-resident inputs; an event pair around every kernel; host buffers
    through less_decode_step_host).  Returns the record of the JSON line (rank 0) or None."""
    import torch
    from paper_2402_09398_b200 import binding, workloads as wl
    dev, world = ranks.dev, ranks.world
    w = wl.CONFIGS[cfg_id]
    if args.batch:
        w = w.with_(batch=args.batch)
    if w.cfg_id == 6:
        cpu_seconds = 0
    if args.group > 1:
        if args.tova or w.heads % args.group:
            raise SystemExit("--group needs a head count it divides and is not defined for --tova")
        w = w.with_(heads=w.heads // args.group, group=args.group)
        cpu_seconds = 0          # context run; the timed oracle leg covers the default workload
    K_steps, W_steps = args.steps, max(args.warmup, 3)
    heavy, recent, flags = w.heavy, w.recent, 0
    if args.full_cache:
        # the cache grows with every step, so the number of steps is fixed in advance
        args.blocks = args.blocks or MIN_BLOCKS
        heavy = w.prompt + W_steps + 2 * K_steps * args.blocks + max(K_steps, 100) + 16
    if args.no_state:
        flags |= binding.LESS_NO_STATE
        heavy += 2 if w.rank == 8 else 4      # Baseline+: slots matching H's storage (Section 4)
        recent += 2 if w.rank == 8 else 4
    if args.lambda_masking:
        flags |= binding.LESS_POLICY_LAMBDA
        heavy, recent = 4, heavy + recent - 4
    if args.tova:
        flags |= binding.LESS_POLICY_TOVA
    if args.out_f16:
        flags |= binding.LESS_OUT_F16
    w_run = w.with_(heavy=heavy, recent=recent)
    out_dtype = torch.float16 if args.out_f16 else torch.float32
    out_bytes = 2 if args.out_f16 else 4

    # replicas: every rank runs the whole workload on its own GPU, no collective in the path
    Wt = wl.make_weights(w, dev)
    layers_per_call = max(1, min(w.layers, (1 << 30) // max(1, w.batch * w.heads * w.group * w.prompt * w.head_dim * 2))) \
        if w.prompt else 1
    ctx = binding.from_workload(w_run, Wt, dev, max_prefill_layers=layers_per_call, flags=flags)
    t_pre0 = time.perf_counter()
    for l0 in range(0, w.layers if w.prompt else 0, layers_per_call):
        n = min(layers_per_call, w.layers - l0)
        Q, Kp, V = wl.make_prompt(w, l0, n, dev)
        ctx.prefill(Q, Kp, V, l0)
        del Q, Kp, V
    if not w.prompt:                       # no prompt phase for this shape: the cache fills by decoding
        ctx.reset()
        fill = [wl.make_decode_inputs(w, s, dev) for s in range(4)]
        for s in range(w_run.slots + 4):
            ctx.decode_step(*fill[s % 4])
        del fill
    torch.cuda.synchronize()
    t_prefill = time.perf_counter() - t_pre0

    # decode inputs of eight steps, resident in HBM before the timed region, used round-robin
    base = [wl.make_decode_inputs(w, s % max(1, w.steps), dev) for s in range(8)]
    out = torch.empty(w.batch, w.layers, w.heads * w.group, w.head_dim, dtype=out_dtype, device=dev)
    stream = torch.cuda.current_stream()
    step_no = [0]

    def one_step():
        q, k, v = base[step_no[0] % len(base)]
        ctx.decode_step(q, k, v, out=out)
        step_no[0] += 1

    for _ in range(W_steps):
        one_step()
    ranks.barrier()
    graph_steps = 0
    if args.graph:
        # 8 consecutive steps, each on its own resident inputs, captured once; the position of every
        # step is read on the device, so each replay continues where the last one stopped
        graph_steps = len(base)
        K_steps = max(graph_steps, K_steps // graph_steps * graph_steps)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for i in range(graph_steps):
                ctx.decode_step(*base[i], out=out)
        stream = torch.cuda.current_stream()

        def run_block():
            for _ in range(K_steps // graph_steps):
                graph.replay()
    else:
        def run_block():
            for _ in range(K_steps):
                one_step()

    # ---- timed region: blocks of K steps, device-resident inputs ----
    sampler = ClockSampler(ranks.local) if ranks.rank == 0 else None
    launches0 = ctx.launches
    t0 = time.time()
    times = timed_blocks(cuda_block_timer(ranks, stream, run_block), ranks.reduce_max, exact_blocks=args.blocks)
    t1 = time.time()
    launches = (ctx.launches - launches0) if not args.graph else 2 * K_steps * len(times)
    clocks = sampler.stop(t0, t1) if sampler else None
    st = block_stats(times, K_steps)

    if args.graph:
        ctx.poll_status()          # the host's copy of the position catches up with the replays
    # ---- the same steps with an event pair around every kernel: per-kernel durations ----
    prof_steps = K_steps if args.blocks else min(max(K_steps, 20), 100)
    ctx.profile(True)
    for _ in range(prof_steps):
        one_step()
    torch.cuda.synchronize()
    prof = ctx.profile_read()
    ctx.profile(False)
    variants = {k: ctx.kernel_variant(k) for k in ("feature_map", "decode")}

    # ---- end to end through the host-buffer entry point ----
    # q and k in one pinned block (k directly behind q: one host-to-device copy), v and the output in
    # pinned memory too (read / written in place by the decode kernel)
    nq_el, nk_el = base[0][0].numel(), base[0][1].numel()
    hqk = torch.empty(nq_el + nk_el, dtype=torch.float16).pin_memory()
    hq, hk = hqk[:nq_el].view(base[0][0].shape), hqk[nq_el:].view(base[0][1].shape)
    hv = torch.empty(base[0][2].shape, dtype=torch.float16).pin_memory()
    hq.copy_(base[0][0]); hk.copy_(base[0][1]); hv.copy_(base[0][2])
    hout = torch.empty(out.shape, dtype=out_dtype).pin_memory()
    for _ in range(3):
        ctx.decode_step_host(hq, hk, hv, hout)

    def e2e_block():
        for _ in range(K_steps):
            ctx.decode_step_host(hq, hk, hv, hout)

    dev_timer = cuda_block_timer(ranks, stream, e2e_block)   # every call synchronises: device time = wall time
    e2e_times = timed_blocks(dev_timer, ranks.reduce_max, min_blocks=5 if not args.blocks else 1,
                             min_total_ms=250.0, exact_blocks=args.blocks)
    st_e2e = block_stats(e2e_times, K_steps)
    status = ctx.poll_status()
    if status != 0:
        raise RuntimeError(f"device status {status} (where-code {ctx.status_where()})")

    rec = None
    if ranks.rank == 0:
        ms_step = st["ms_per_step"]
        units = w.instances * w.group
        value = units * world / (ms_step * 1e-3)
        e2e_value = units * world / (st_e2e["ms_per_step"] * 1e-3)
        peak, _, peak_kind = peaks()
        n_live = min(w_run.slots, w.prompt + W_steps) if w.prompt else w_run.slots
        evicting = not args.full_cache
        kb = {"feature_map": feature_map_bytes(w, args.no_state),
              "decode": decode_bytes(w, n_live, evicting, args.no_state, out_bytes)}
        kt = {k: (prof[k][0] / prof[k][1] if prof[k][1] else 0.0) for k in ("feature_map", "decode")}
        if kt["feature_map"] == 0.0 and kb["feature_map"]:      # a step of one launch: the maps' bytes move in it
            kb = {"feature_map": 0, "decode": kb["feature_map"] + kb["decode"]}
        dominant = max(kt, key=lambda k: kt[k])
        ach = kb[dominant] / (kt[dominant] * 1e-3) / 1e9 if kt[dominant] > 0 else 0.0
        step_bytes = kb["feature_map"] + kb["decode"]
        step_gbs = step_bytes / (ms_step * 1e-3) / 1e9
        narrow = kv_state_scores_bytes(w, n_live, args.no_state)
        narrow_gbs = narrow / (ms_step * 1e-3) / 1e9
        wl_key = f"cfg{w.cfg_id}" + (f"_b{w.batch}" if args.batch else "") + (f"_g{w.group}" if w.group > 1 else "")
        traffic, traffic_note = ncu_traffic(wl_key, dominant)
        rec = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K_steps,
            "warmup": W_steps, "ms_per_step": ms_step, "ms_per_step_min": st["ms_per_step_min"],
            "blocks": st["blocks"], "timed_device_ms": st["timed_device_ms"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(w, args),
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT,
                    "h2d_bytes_per_step": (2 + w.group) * w.instances * w.head_dim * 2,
                    "d2h_bytes_per_step": w.group * w.instances * w.head_dim * out_bytes,
                    "ms_per_step": st_e2e["ms_per_step"], "ms_per_step_min": st_e2e["ms_per_step_min"],
                    "blocks": st_e2e["blocks"]},
            "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "kernel": variants[dominant], "achieved": ach, "peak": peak,
                         "unit": "GB/s", "frac": ach / peak, "peak_kind": f"of {peak_kind}",
                         "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS,
                         "traffic": traffic, "traffic_note": traffic_note,
                         "algorithmic_bytes_per_launch": kb[dominant],
                         "kernels": variants,
                         "kernel_us": {k: 1e3 * v for k, v in kt.items()},
                         "kernel_GBs": {k: (kb[k] / (kt[k] * 1e-3) / 1e9 if kt[k] > 0 else 0.0) for k in kt},
                         "step_algorithmic_bytes": step_bytes, "step_GBs": step_gbs,
                         "step_frac": step_gbs / peak, "step_frac_of_nominal_8TBs": step_gbs / NOMINAL_HBM_GBS,
                         "kv_state_scores_bytes": narrow, "kv_state_scores_GBs": narrow_gbs,
                         "kv_state_scores_frac": narrow_gbs / peak,
                         "kv_state_scores_frac_of_nominal_8TBs": narrow_gbs / NOMINAL_HBM_GBS},
            "prefill_s": t_prefill,
        }
        if cpu_seconds > 0 and world == 1:
            instances = list(range(0, w.instances, max(1, w.instances // 16)))[:16]
            recs = ctx.export_state(instances)
            Wc = {k: v.cpu() for k, v in Wt.items()}
            rate, cores, sample, _, _ = oracle_rate(w, cpu_seconds, recs, instances, Wc)
            rec["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}
    ctx.close()
    del ctx, base, out, Wt
    torch.cuda.empty_cache()
    return rec


# --------------------------------------------------------------------------- #
# prompt compression (workload 5): a step = the prompt phase of one layer
# --------------------------------------------------------------------------- #
def prefill_flops(w):
    """Algorithmic flops of one layer's prompt phase, per kernel (fp16 inputs, fp32 accumulate)."""
    inst = w.batch * w.heads
    S, D, Rp, R = w.prompt, w.head_dim, w.hidden, w.rank
    causal = S * (S + 1) // 2
    qh = inst * w.group                    # the scoring kernels work per query head
    return {"rowstat": qh * causal * 2 * D, "colsum": qh * causal * 2 * D, "attn_out": qh * causal * 4 * D,
            "psi": inst * S * 2 * (D * Rp + Rp * R + R * R), "build": inst * S * 2 * R * D}


def measure_prefill(args, ranks, cpu_seconds, steps=None):
    import torch
    from paper_2402_09398_b200 import binding, workloads as wl
    dev, world = ranks.dev, ranks.world
    w = wl.CONFIGS[5]
    if args.batch:
        w = w.with_(batch=args.batch)
    if args.group > 1:
        w = w.with_(heads=w.heads // args.group, group=args.group)
    K_steps, W_steps = steps or args.steps, max(args.warmup, 3)
    Wt = wl.make_weights(w, dev)
    ctx = binding.from_workload(w, Wt, dev, max_prefill_layers=1)
    Q, Kp, V = wl.make_prompt(w, 0, 1, dev)          # one layer of inputs, reused for every layer index
    attn = torch.empty(Q.shape, dtype=torch.float32, device=dev) if args.attn_out else None
    stream = torch.cuda.current_stream()
    step_no = [0]

    def one_step():
        ctx.prefill(Q, Kp, V, step_no[0] % w.layers, attn_out=attn)
        step_no[0] += 1

    def run_block():
        for _ in range(K_steps):
            one_step()

    for _ in range(W_steps):
        one_step()
    ranks.barrier()
    sampler = ClockSampler(ranks.local) if ranks.rank == 0 else None
    launches0 = ctx.launches
    t0 = time.time()
    times = timed_blocks(cuda_block_timer(ranks, stream, run_block), ranks.reduce_max, exact_blocks=args.blocks)
    t1 = time.time()
    launches = ctx.launches - launches0
    clocks = sampler.stop(t0, t1) if sampler else None
    st = block_stats(times, K_steps)
    ctx.profile(True)
    for _ in range(max(K_steps, 3) if not args.blocks else K_steps):
        one_step()
    torch.cuda.synchronize()
    prof = ctx.profile_read()
    ctx.profile(False)
    variants = {k: ctx.kernel_variant(k) for k in ("rowstat", "colsum", "attn_out", "select", "psi", "gather", "build", "finalize")}
    # end to end: the layer's Q, K, V come from pinned host memory, the kept positions go back
    hq, hk, hv = (torch.empty(t.shape, dtype=torch.float16).pin_memory() for t in (Q, Kp, V))
    hq.copy_(Q); hk.copy_(Kp); hv.copy_(V)
    dq, dk, dv = torch.empty_like(Q), torch.empty_like(Kp), torch.empty_like(V)
    inst0 = list(range(0, w.batch * w.layers * w.heads, w.layers * w.heads))[:w.batch]
    torch.cuda.synchronize()
    tw0 = time.perf_counter()
    n_e2e = 2 if not args.blocks else 1
    for _ in range(n_e2e):
        dq.copy_(hq, non_blocking=True); dk.copy_(hk, non_blocking=True); dv.copy_(hv, non_blocking=True)
        ctx.prefill(dq, dk, dv, step_no[0] % w.layers)
        step_no[0] += 1
        ctx.export_state(inst0[:1])                    # device -> host read of one instance's kept set
    torch.cuda.synchronize()
    ms_e2e = 1e3 * (time.perf_counter() - tw0) / n_e2e
    status = ctx.poll_status()
    if status != 0:
        raise RuntimeError(f"device status {status} (where-code {ctx.status_where()})")
    ms_e2e = ranks.reduce_max([ms_e2e])[0]
    rec = None
    if ranks.rank == 0:
        ms_step = st["ms_per_step"]
        tokens = w.batch * w.heads * w.group * w.prompt * world
        fl = prefill_flops(w)
        kt = {k: (prof[k][0] / prof[k][1] if prof[k][1] else 0.0) for k in prof}
        dominant = max(fl, key=lambda k: kt.get(k, 0.0))
        _, peak, kind = peaks()
        kind = f"of {kind} (sustained bf16 = fp16 rate)"
        ach = fl[dominant] / (kt[dominant] * 1e-3) / 1e12 if kt.get(dominant) else 0.0

        def part(keys):
            ms = sum(kt.get(k, 0.0) for k in keys)
            f = sum(fl[k] for k in keys if k in fl and kt.get(k, 0.0) > 0)
            tf = f / (ms * 1e-3) / 1e12 if ms else 0.0
            return {"ms": ms, "algorithmic_flops": f, "TFLOPs": tf, "frac": tf / peak}
        rec = {"metric": PROMPT_METRIC,
               "value": tokens / (ms_step * 1e-3), "unit": "head-tokens/s", "n_gpus": world, "steps": K_steps,
               "warmup": W_steps, "ms_per_step": ms_step, "ms_per_step_min": st["ms_per_step_min"],
               "blocks": st["blocks"], "timed_device_ms": st["timed_device_ms"],
               "higher_is_better": True, "scaling": "weak",
               "vs_baseline": None, "dtype": "f16 inputs, f32 accumulate", "data": "synthetic",
               "config": {"workload": workload_name(w, args)
                          + (f" [grouped query heads: {w.heads} KV heads x {w.group}; the unit counts query heads]"
                             if w.group > 1 else ""),
                          "instances_per_step": w.batch * w.heads,
                          "l2": "6.3 GB of Q, K, V per step exceed the 126 MB L2"},
               "clocks": clocks,
               "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": "head-tokens/s",
                       "h2d_bytes_per_step": (Q.numel() + Kp.numel() + V.numel()) * 2,
                       "d2h_bytes_per_step": ctx.record_bytes},
               "gpu_launches": int(launches),
               "roofline": {"bound": "tensor", "kernel": variants.get(dominant) or dominant, "achieved": ach, "peak": peak,
                            "unit": "TFLOP/s", "frac": ach / peak, "peak_kind": kind, "traffic": None,
                            "algorithmic_flops_per_launch": fl[dominant],
                            "kernels": {k: v for k, v in variants.items() if v},
                            "kernel_ms": {k: v for k, v in kt.items() if v},
                            "kernel_TFLOPs": {k: fl[k] / (kt[k] * 1e-3) / 1e12 for k in fl if kt.get(k)},
                            # the two halves of the prompt phase, each against the same dense peak
                            "scoring": part(["rowstat", "colsum", "attn_out"]),
                            "state_build": part(["psi", "build", "finalize"])}}
        if cpu_seconds > 0 and world == 1:
            rate, cores, sample = oracle_prompt_rate(w, 2048, cpu_seconds)
            rec["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}
    ctx.close()
    del ctx, Q, Kp, V, dq, dk, dv, hq, hk, hv, Wt
    torch.cuda.empty_cache()
    return rec


def measure_masked(args, ranks):
    """The parallel form: a step = less_masked_attention over one layer (B x heads sequences)."""
    import torch
    from paper_2402_09398_b200 import binding, workloads as wl
    dev, world = ranks.dev, ranks.world
    S = args.seq
    w = wl.CONFIGS[2].with_(batch=args.batch or 2, prompt=S, heavy=int(0.05 * S), recent=int(0.05 * S))
    if args.group > 1:                                   # the same query heads over fewer KV heads
        w = w.with_(heads=w.heads // args.group, group=args.group)
    K_steps, W_steps = args.steps, max(args.warmup, 3)
    Wt = wl.make_weights(w, dev)
    ctx = binding.from_workload(w, Wt, dev, max_prefill_layers=1, flags=binding.LESS_WITH_PARALLEL_FORM)
    Q, Kp, V = wl.make_prompt(w, 0, 1, dev)
    # schedule: every key leaves between `recent` and `recent + 2 * slots` steps after its own
    gen = torch.Generator(device=dev).manual_seed(1234)
    pos = torch.arange(S, device=dev).expand(w.batch, 1, w.heads, S)
    eu = (pos + w.recent + torch.randint(0, 2 * w.slots, pos.shape, generator=gen, device=dev)).to(torch.int32).contiguous()
    out = torch.empty(Q.shape, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    step_no = [0]

    def one_step():
        ctx.masked_attention(Q, Kp, V, eu, layer_begin=step_no[0] % w.layers, out=out)
        step_no[0] += 1

    def run_block():
        for _ in range(K_steps):
            one_step()

    for _ in range(W_steps):
        one_step()
    ranks.barrier()
    sampler = ClockSampler(ranks.local) if ranks.rank == 0 else None
    launches0 = ctx.launches
    t0 = time.time()
    times = timed_blocks(cuda_block_timer(ranks, stream, run_block), ranks.reduce_max, exact_blocks=args.blocks)
    t1 = time.time()
    launches = ctx.launches - launches0
    clocks = sampler.stop(t0, t1) if sampler else None
    st = block_stats(times, K_steps)
    ctx.profile(True)
    for _ in range(K_steps):
        one_step()
    torch.cuda.synchronize()
    prof = ctx.profile_read()
    ctx.profile(False)
    # end to end: inputs from pinned host memory, the output read back
    hq, hk, hv = (torch.empty(t.shape, dtype=torch.float16).pin_memory() for t in (Q, Kp, V))
    heu = torch.empty(eu.shape, dtype=torch.int32).pin_memory()
    hq.copy_(Q); hk.copy_(Kp); hv.copy_(V); heu.copy_(eu)
    hout = torch.empty(out.shape, dtype=torch.float32).pin_memory()
    dq, dk, dv, deu = torch.empty_like(Q), torch.empty_like(Kp), torch.empty_like(V), torch.empty_like(eu)
    torch.cuda.synchronize()
    tw0 = time.perf_counter()
    n_e2e = max(1, min(K_steps, 3))
    for _ in range(n_e2e):
        dq.copy_(hq, non_blocking=True); dk.copy_(hk, non_blocking=True); dv.copy_(hv, non_blocking=True)
        deu.copy_(heu, non_blocking=True)
        ctx.masked_attention(dq, dk, dv, deu, layer_begin=0, out=out)
        hout.copy_(out, non_blocking=True)
    torch.cuda.synchronize()
    ms_e2e = 1e3 * (time.perf_counter() - tw0) / n_e2e
    status = ctx.poll_status()
    if status != 0:
        raise RuntimeError(f"device status {status} (where-code {ctx.status_where()})")
    ms_e2e = ranks.reduce_max([ms_e2e])[0]
    rec = None
    if ranks.rank == 0:
        ms_step = st["ms_per_step"]
        inst = w.batch * w.heads * w.group               # sequences of query rows
        tokens = inst * S * world
        # flops of the entries the kernel has to form: 128 x 128 tiles that are not dead (a key tile all of
        # whose keys were discarded before a Q tile's first row is handled through its summed state)
        nt = (S + 127) // 128
        eu_pad = torch.full((w.batch, 1, w.heads, nt * 128), 0, dtype=torch.int64, device=dev)
        eu_pad[..., :S] = eu.long()
        death = eu_pad.view(w.batch, 1, w.heads, nt, 128).amax(-1)
        first_dead = torch.maximum((death + 127) // 128, torch.arange(nt, device=dev) + 1).clamp(max=nt)
        live_pairs = int((first_dead - torch.arange(nt, device=dev)).sum().item()) * w.group
        live_frac = live_pairs / (inst * nt * (nt + 1) / 2)
        fl = {"masked_out": live_pairs * 128 * 128 * (4 * w.head_dim + 2 * w.rank),
              "psi": (inst + w.batch * w.heads) * S * (2 * w.head_dim * w.hidden + 2 * w.hidden * w.rank + w.rank * w.rank)}
        kt = {k: (prof[k][0] / prof[k][1] if prof[k][1] else 0.0) for k in prof}
        kt["psi"] *= 2                                   # psi and phi launches are booked under the same id
        kt["masked_pack"] *= 3                           # operand pack, tile states, running sums
        dominant = max(fl, key=lambda k: kt.get(k, 0.0))
        _, peak, kind = peaks()
        kind = f"of {kind} (sustained bf16 = fp16 rate)"
        ach = fl[dominant] / (kt[dominant] * 1e-3) / 1e12 if kt.get(dominant) else 0.0
        rec = {"metric": "parallel-form head-tokens/s (one layer per step)", "value": tokens / (ms_step * 1e-3),
               "unit": "head-tokens/s", "n_gpus": world, "steps": K_steps, "warmup": W_steps, "ms_per_step": ms_step,
               "ms_per_step_min": st["ms_per_step_min"], "blocks": st["blocks"],
               "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
               "dtype": "f16 inputs, f32 accumulate", "data": "synthetic",
               "config": {"workload": f"parallel form (B={w.batch}, {w.heads * w.group} query heads"
                                      + (f" over {w.heads} KV heads" if w.group > 1 else "")
                                      + f", sequences of {S}, one layer per step, R={w.rank})",
                          "instances_per_step": inst, "live_tile_fraction": live_frac, "l2": "inputs, operands and output of a step exceed the 126 MB L2"
                          if inst * S * 1300 > 126e6 else "a step's data fit the L2"},
               "clocks": clocks,
               "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": "head-tokens/s",
                       "h2d_bytes_per_step": (Q.numel() + 2 * Kp.numel()) * 2 + eu.numel() * 4,
                       "d2h_bytes_per_step": out.numel() * 4},
               "gpu_launches": int(launches),
               "roofline": {"bound": "tensor", "kernel": "masked_out_tc_kernel" if dominant == "masked_out" else dominant,
                            "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak, "peak_kind": kind,
                            "traffic": None, "algorithmic_flops_per_launch": fl[dominant],
                            "kernel_ms": {k: v for k, v in kt.items() if v}}}
    ctx.close()
    return rec


SUB_RECORD_KEYS = ("metric", "value", "unit", "steps", "warmup", "ms_per_step", "ms_per_step_min", "blocks",
                   "timed_device_ms", "dtype", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline",
                   "prefill_s")


def run_b200(args):
    from paper_2402_09398_b200 import binding, build
    ranks = Ranks()
    build.build()
    binding.lib()
    if args.masked_form:
        line = measure_masked(args, ranks)
    elif args.config == 5:
        line = measure_prefill(args, ranks, 0 if args.no_cpu_baseline else args.cpu_seconds)
    elif args.config:
        line = measure_decode(args, ranks, args.config, 0 if args.no_cpu_baseline else args.cpu_seconds)
    else:
        # the headline, then the other workloads as sub-records (a failure there is recorded, not fatal)
        line = measure_decode(args, ranks, HEADLINE_CONFIG, 0 if args.no_cpu_baseline else args.cpu_seconds)
        subs = {}
        short = 0 if args.no_cpu_baseline else min(3.0, args.cpu_seconds)
        for cfg in (1, 2, 4, 5):
            try:
                r = measure_prefill(args, ranks, short, steps=1) if cfg == 5 else measure_decode(args, ranks, cfg, short)
            except Exception as e:                    # noqa: BLE001 - reported in the line
                r = {"error": repr(e)}
                if ranks.world > 1:
                    raise
            if ranks.rank == 0:
                subs[f"cfg{cfg}"] = {k: r[k] for k in SUB_RECORD_KEYS if k in r} if "error" not in r else r
        # context: the same decode kernel over a full cache (nothing evicted) and with the sparse policy
        # alone (Baseline+), on the batch-1 Llama-2-7B shape
        import copy
        context = {}
        for name, kw in (("cfg2_full_cache", {"full_cache": True}), ("cfg2_baseline_plus", {"no_state": True})):
            a = copy.copy(args)
            for k, v in kw.items():
                setattr(a, k, v)
            try:
                r = measure_decode(a, ranks, 2, 0)
            except Exception as e:                    # noqa: BLE001 - reported in the line
                r = {"error": repr(e)}
                if ranks.world > 1:
                    raise
            if ranks.rank == 0:
                context[name] = {k: r[k] for k in SUB_RECORD_KEYS if k in r} if "error" not in r else r
        if ranks.rank == 0:
            line["configs"] = subs
            line["context"] = context
    if ranks.rank == 0:
        print(json.dumps(line))
    ranks.close()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(launch_ranks(args.gpus, os.path.abspath(__file__), sys.argv[1:]))
    if args.gpus != int(os.environ.get("WORLD_SIZE", "1")):
        raise SystemExit(f"--gpus {args.gpus} does not match WORLD_SIZE={os.environ.get('WORLD_SIZE')}")
    run_b200(args)


if __name__ == "__main__":
    main()
