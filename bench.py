#!/usr/bin/env python
"""Benchmark of the LESS decode hot path on B200.

A step = one generation step (Algorithm 1) of every (batch, layer, head)
instance of the workload: feature maps, attention over the kept slots with the
low-rank correction, score update, eviction, state update.  The cache is first
built by the library's own prompt phase from seeded synthetic Q/K/V, then
`--warmup` untimed and `--steps` timed decode steps run.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl reference]

Prints ONE JSON line (rank 0).  With --impl reference the fp64 CPU oracle is
timed instead, on a bounded sample of the same workload.
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

METRIC = "decode attention head-tokens/s (B x layers x heads per step)"
UNIT = "head-tokens/s"
FALLBACK_HBM_GBS = 6650.0

# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures
# summarised under profiles/ (None where no capture of that kernel and workload exists)
NCU_TRAFFIC_BYTES = {
    (2, "feature_map"): 285.91e6 + 6.29e6,   # profiles/decode_step_cfg2.md
    (2, "decode"): 113.88e6 + 3.77e6,
    # cfg3 captured at batch 16 (a quarter of the instances): the decode kernel's traffic is per
    # instance and scales by 4; the feature maps' weight traffic does not scale and is not listed
    (3, "decode"): 4 * (1.824e9 + 56.1e6),
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", type=int, default=2, help="workload id (1-4 decode; 5 = prompt compression, one layer per step)")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="budget of the CPU-baseline leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
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
    return ap.parse_args()


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


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


def decode_bytes(w, n_live, evicting=True, no_state=False):
    D, R, G = w.head_dim, w.rank, w.group
    per = n_live * (2 * D * 2)              # K and V rows
    per += n_live * (4 + 4)                 # accumulated score read + write
    per += n_live * 4 if evicting else 0    # positions (only read when a victim is needed)
    per += (2 + G) * D * 2 + G * D * 4      # q, k, v in; out (G query heads per KV head)
    per += 2 * D * 2 + 8                    # new pair into its slot, pos, acc
    per += 4                                # slot count
    if not no_state:
        per += R * D * 4 + R * 4            # H, z read
        per += (G + 1) * R * 4              # phi(q) of the G heads, psi(k) read
        per += R * 4                        # psi into the slot's cache
        if evicting:
            per += R * D * 4 + R * 4 + R * 4 + D * 2   # H, z write; victim psi; victim v row
    return w.instances * per


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


class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML (read-only) every
    10 ms on a thread while the timed region runs."""

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
            time.sleep(0.01)

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
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": self.max_mhz,
                "reasons": reasons, "samples": len(sm)}


# --------------------------------------------------------------------------- #
# CPU oracle timing (cpu_baseline leg and --impl reference)
# --------------------------------------------------------------------------- #
def oracle_rate(w, seconds, records=None, instances=None, W=None, max_instances=16):
    """Times oracle decode steps on a bounded sample of instances.  With
    `records` (states exported from the GPU) the oracle starts from them, else it
    runs its own prompt phase first (untimed).  Returns (head-tokens/s, cores, text)."""
    import numpy as np
    from threadpoolctl import threadpool_limits
    from oracle import less_oracle as lo
    from paper_2402_09398_b200 import workloads as wl
    if W is None:
        W = wl.make_weights(w, "cpu")
    with threadpool_limits(limits=1):
        if instances is None:
            instances = list(range(0, w.instances, max(1, w.instances // max_instances)))[:max_instances]
        orcs = []
        prompt_cache = {}
        for n, inst in enumerate(instances):
            b, layer, head = wl.instance_coords(w, inst)
            wts = [W[k][layer, head].double().cpu().numpy() for k in
                   ("w_phi1", "w_phi2", "w_psi1", "w_psi2", "w_psi3")]
            o = lo.LessInstance(w.head_dim, w.rank, w.heavy, w.recent, *lo.make_mlp_maps(*wts))
            if records is not None:
                r = records[n]
                o.import_state(r["pos"], r["K"], r["V"], r["acc"], r["H"], r["z"], r["t"])
            else:
                if layer not in prompt_cache:
                    prompt_cache = {layer: wl.make_prompt(w, layer, 1, "cpu")}
                Q, K, V = prompt_cache[layer]
                o.prefill(*(t[b, 0, head].double().numpy() for t in (Q, K, V)))
            orcs.append(o)
        units, t_used, step = 0, 0.0, 0
        while t_used < seconds and step < max(w.steps, 1):
            q, k, v = wl.make_decode_inputs(w, step, "cpu")
            q, k, v = (t.reshape(-1, w.head_dim).double().numpy() for t in (q, k, v))
            t0 = time.perf_counter()
            for inst, o in zip(instances, orcs):
                o.decode(q[inst], k[inst], v[inst])
            t_used += time.perf_counter() - t0
            units += len(instances)
            step += 1
    sample = (f"{len(instances)} of {w.instances} instances x {step} decode steps "
              f"({'GPU-exported' if records is not None else 'oracle-prefilled'} state), fp64 numpy, 1 thread")
    return units / t_used, 1, sample, step, t_used


def run_reference(args):
    from paper_2402_09398_b200 import workloads as wl
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = wl.CONFIGS[args.config]
    # each "step" = one oracle decode step over the sampled instances
    per_step_budget = 120.0 / max(1, args.steps + args.warmup)
    n_inst = 8
    w_run = w.with_(steps=args.steps + args.warmup)
    rate, cores, sample, steps_done, t_used = oracle_rate(
        w_run, seconds=per_step_budget * (args.steps + args.warmup), max_instances=n_inst)
    line = {
        "impl": "reference", "metric": METRIC, "value": rate, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_used / max(1, steps_done),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(w, args),
        "cpu_baseline": {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": rate, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(w, args):
    name = {1: "cfg1 smallest (B=1, 1 layer x 8 heads, prompt 256, 32+32 slots, R=8)",
            2: "cfg2 Llama-2-7B shape (B=1, 32 layers x 32 heads, prompt 2048, 102+102 slots, R=8)",
            3: "cfg3 batched serving (B=64, 32 layers x 32 heads, prompt 1024, 102+102 slots, R=8)",
            4: "cfg4 long context (B=4, 40 layers x 40 heads, prompt 16384, 327+327 slots, R=16)"}[w.cfg_id]
    if getattr(args, "batch", 0):
        name += f" [batch set to {w.batch} for profiling]"
    c = {"workload": name, "instances": w.instances, "slots": w.slots, "rank": w.rank,
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
    return c


# --------------------------------------------------------------------------- #
def run_b200(args):
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2402_09398_b200 import binding, build, workloads as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the LESS path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
    build.build()
    binding.lib()

    w = wl.CONFIGS[args.config]
    if args.batch:
        w = w.with_(batch=args.batch)
    if args.group > 1:
        if args.tova or w.heads % args.group:
            raise SystemExit("--group needs a head count it divides and is not defined for --tova")
        w = w.with_(heads=w.heads // args.group, group=args.group)
        args.no_cpu_baseline = True      # context run; the timed oracle leg covers the default workload
    K_steps, W_steps = args.steps, args.warmup
    total_steps = K_steps * 3 + W_steps + 2
    heavy, recent, flags = w.heavy, w.recent, 0
    if args.full_cache:
        heavy = w.prompt + total_steps
    if args.no_state:
        flags |= binding.LESS_NO_STATE
        heavy += 2 if w.rank == 8 else 4      # Baseline+: slots matching H's storage (Section 4)
        recent += 2 if w.rank == 8 else 4
    if args.lambda_masking:
        flags |= binding.LESS_POLICY_LAMBDA
        heavy, recent = 4, heavy + recent - 4
    if args.tova:
        flags |= binding.LESS_POLICY_TOVA
    w_run = w.with_(heavy=heavy, recent=recent)

    # replicas: every rank runs the whole workload on its own GPU, no collective in the path
    Wt = wl.make_weights(w, dev)
    layers_per_call = max(1, min(w.layers, (1 << 30) // max(1, w.batch * w.heads * w.group * w.prompt * w.head_dim * 2)))
    ctx = binding.from_workload(w_run, Wt, dev, max_prefill_layers=layers_per_call, flags=flags)
    t_pre0 = time.perf_counter()
    for l0 in range(0, w.layers, layers_per_call):
        n = min(layers_per_call, w.layers - l0)
        Q, Kp, V = wl.make_prompt(w, l0, n, dev)
        ctx.prefill(Q, Kp, V, l0)
        del Q, Kp, V
    torch.cuda.synchronize()
    t_prefill = time.perf_counter() - t_pre0

    # decode inputs for every step, resident in HBM before the timed region
    inputs = [wl.make_decode_inputs(w, s % max(1, w.steps), dev) if s < 8 else None for s in range(total_steps)]
    base = [i for i in inputs if i is not None]
    inputs = [base[s % len(base)] for s in range(total_steps)]
    out = torch.empty(w.batch, w.layers, w.heads * w.group, w.head_dim, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    step_no = [0]

    def one_step():
        q, k, v = inputs[step_no[0] % total_steps]
        ctx.decode_step(q, k, v, out=out)
        step_no[0] += 1

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(W_steps, 3)):
        one_step()
    barrier()
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

        def run_steps(n):
            for _ in range(n // graph_steps):
                graph.replay()
    else:
        def run_steps(n):
            for _ in range(n):
                one_step()

    # ---- timed region: K steps, device-resident inputs ----
    sampler = ClockSampler(local) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ctx.launches
    barrier()
    t0 = time.time()
    e0.record(stream)
    run_steps(K_steps)
    e1.record(stream)
    barrier()
    t1 = time.time()
    launches = (ctx.launches - launches0) if not args.graph else 2 * K_steps
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop(t0, t1) if sampler else None

    if args.graph:
        ctx.poll_status()          # the host's copy of the position catches up with the replays
    # ---- same K steps with an event pair around every kernel: per-kernel durations ----
    ctx.profile(True)
    for _ in range(K_steps):
        one_step()
    torch.cuda.synchronize()
    prof = ctx.profile_read()
    ctx.profile(False)

    # ---- end to end through the host-buffer entry point ----
    hq, hk, hv = (torch.empty(inputs[0][i].shape, dtype=torch.float16).pin_memory() for i in range(3))
    hq.copy_(inputs[0][0]); hk.copy_(inputs[0][1]); hv.copy_(inputs[0][2])
    hout = torch.empty(out.shape, dtype=torch.float32).pin_memory()
    for _ in range(3):
        ctx.decode_step_host(hq, hk, hv, hout)
    barrier()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record(stream)
    tw0 = time.perf_counter()
    for _ in range(K_steps):
        ctx.decode_step_host(hq, hk, hv, hout)
    e3.record(stream)
    torch.cuda.synchronize()
    ms_e2e = max(e2.elapsed_time(e3), 1e3 * (time.perf_counter() - tw0))
    status = ctx.poll_status()
    if status != 0:
        raise RuntimeError(f"device status {status}")

    ms, ms_e2e = max_over_ranks([ms, ms_e2e], dev, world)

    if rank == 0:
        value = job_throughput(w.instances * w.group, K_steps, ms, world)
        e2e_value = job_throughput(w.instances * w.group, K_steps, ms_e2e, world)
        peak, peak_kind = peaks()
        n_live = min(w_run.slots, w.prompt + W_steps)
        evicting = not args.full_cache
        kb = {"feature_map": feature_map_bytes(w, args.no_state),
              "decode": decode_bytes(w, n_live, evicting, args.no_state)}
        kt = {k: (prof[k][0] / prof[k][1] if prof[k][1] else 0.0) for k in ("feature_map", "decode")}
        dominant = max(kt, key=lambda k: kt[k])
        kernel_names = {"feature_map": ("feature_tc_small_kernel" if w.batch <= 8 else "feature_tc_kernel")
                        + f"<{w.rank}" + (f", {1 if w.batch <= 1 else 2 if w.batch <= 2 else 4 if w.batch <= 4 else 8}>"
                                          if w.batch <= 8 else ">"),
                        "decode": (f"decode_kernel<{w.rank}, {1 if args.graph else 0}>" if w.group == 1 else
                                   f"decode_group_mma_kernel<{w.rank}, {w.group}, {1 if args.graph else 0}>")}
        ach = kb[dominant] / (kt[dominant] * 1e-3) / 1e9 if kt[dominant] > 0 else 0.0
        step_bytes = kb["feature_map"] + kb["decode"]
        kv_state_bytes = w.instances * (n_live * (4 * w.head_dim + 8) + (0 if args.no_state else 2 * w.rank * w.head_dim * 4))
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K_steps,
            "warmup": max(W_steps, 3), "ms_per_step": ms / K_steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(w, args),
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT,
                    "h2d_bytes_per_step": (2 + w.group) * w.instances * w.head_dim * 2,
                    "d2h_bytes_per_step": w.group * w.instances * w.head_dim * 4},
            "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "kernel": kernel_names[dominant], "achieved": ach, "peak": peak,
                         "unit": "GB/s", "frac": ach / peak, "peak_kind": f"of {peak_kind}",
                         "frac_of_nominal_8TBs": ach / 8000.0,
                         "traffic": NCU_TRAFFIC_BYTES.get((w.cfg_id, dominant)),
                         "algorithmic_bytes_per_launch": kb[dominant],
                         "kernel_us": {k: 1e3 * v for k, v in kt.items()},
                         "kernel_GBs": {k: (kb[k] / (kt[k] * 1e-3) / 1e9 if kt[k] > 0 else 0.0) for k in kt},
                         "step_algorithmic_bytes": step_bytes,
                         "step_GBs": step_bytes / (ms / K_steps * 1e-3) / 1e9,
                         "step_frac": step_bytes / (ms / K_steps * 1e-3) / 1e9 / peak,
                         "kv_state_scores_GBs": kv_state_bytes / (ms / K_steps * 1e-3) / 1e9},
            "prefill_s": t_prefill,
        }
        if not args.no_cpu_baseline and world == 1:
            instances = list(range(0, w.instances, max(1, w.instances // 16)))[:16]
            recs = ctx.export_state(instances)
            Wc = {k: v.cpu() for k, v in Wt.items()}
            rate, cores, sample, _, _ = oracle_rate(w.with_(steps=max(w.steps, 64)), args.cpu_seconds, recs, instances, Wc)
            line["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": sample}
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()



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


def run_prefill(args):
    import torch
    import torch.distributed as dist
    from paper_2402_09398_b200 import binding, build, workloads as wl
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the LESS path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
    build.build()
    w = wl.CONFIGS[args.config]
    if args.batch:
        w = w.with_(batch=args.batch)
    if args.group > 1:
        w = w.with_(heads=w.heads // args.group, group=args.group)
    K_steps, W_steps = args.steps, max(args.warmup, 3)
    Wt = wl.make_weights(w, dev)
    ctx = binding.from_workload(w, Wt, dev, max_prefill_layers=1)
    Q, Kp, V = wl.make_prompt(w, 0, 1, dev)          # one layer of inputs, reused for every layer index
    attn = torch.empty(Q.shape, dtype=torch.float32, device=dev) if args.attn_out else None
    stream = torch.cuda.current_stream()
    step_no = [0]

    def one_step():
        ctx.prefill(Q, Kp, V, step_no[0] % w.layers, attn_out=attn)
        step_no[0] += 1

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(W_steps):
        one_step()
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ctx.launches
    t0 = time.time()
    e0.record(stream)
    for _ in range(K_steps):
        one_step()
    e1.record(stream)
    barrier()
    t1 = time.time()
    launches = ctx.launches - launches0
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop(t0, t1) if sampler else None
    ctx.profile(True)
    for _ in range(K_steps):
        one_step()
    torch.cuda.synchronize()
    prof = ctx.profile_read()
    ctx.profile(False)
    # end to end: the layer's Q, K, V come from pinned host memory, the kept positions go back
    hq, hk, hv = (torch.empty(t.shape, dtype=torch.float16).pin_memory() for t in (Q, Kp, V))
    hq.copy_(Q); hk.copy_(Kp); hv.copy_(V)
    dq, dk, dv = torch.empty_like(Q), torch.empty_like(Kp), torch.empty_like(V)
    inst0 = list(range(0, w.batch * w.layers * w.heads, w.layers * w.heads))[:w.batch]
    torch.cuda.synchronize()
    tw0 = time.perf_counter()
    n_e2e = max(1, min(K_steps, 3))
    for _ in range(n_e2e):
        dq.copy_(hq, non_blocking=True); dk.copy_(hk, non_blocking=True); dv.copy_(hv, non_blocking=True)
        ctx.prefill(dq, dk, dv, step_no[0] % w.layers)
        step_no[0] += 1
        ctx.export_state(inst0[:1])                    # device -> host read of one instance's kept set
    torch.cuda.synchronize()
    ms_e2e = 1e3 * (time.perf_counter() - tw0) / n_e2e
    if ctx.poll_status() != 0:
        raise RuntimeError("device status")
    ms, ms_e2e = max_over_ranks([ms, ms_e2e], dev, world)
    if rank == 0:
        tokens = w.batch * w.heads * w.group * w.prompt * world
        fl = prefill_flops(w)
        kt = {k: (prof[k][0] / prof[k][1] if prof[k][1] else 0.0) for k in prof}
        dominant = max(fl, key=lambda k: kt.get(k, 0.0))
        p = os.path.join(ROOT, "MEASURED_PEAKS.json")
        peak, kind = (float(json.load(open(p))["bf16_tflops_sustained"]), "of measured (sustained bf16 = fp16 rate)") \
            if os.path.exists(p) else (1400.0, "of fallback")
        ach = fl[dominant] / (kt[dominant] * 1e-3) / 1e12 if kt.get(dominant) else 0.0
        rec_bytes = ctx.record_bytes if hasattr(ctx, "record_bytes") else None
        line = {"metric": "prompt head-tokens/s (prompt scoring, selection, state build; one layer per step)",
                "value": tokens * K_steps / (ms * 1e-3), "unit": "head-tokens/s", "n_gpus": world, "steps": K_steps,
                "warmup": W_steps, "ms_per_step": ms / K_steps, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f16 inputs, f32 accumulate", "data": "synthetic",
                "config": {"workload": f"cfg5 prefill compression (B={w.batch}, 32 heads, one layer per step, "
                                       "prompt 32768, 1638+1638 slots, R=16)"
                                       + (" [batch reduced for profiling]" if args.batch else "")
                                       + (f" [grouped query heads: {w.heads} KV heads x {w.group}; the unit counts query heads]"
                                          if w.group > 1 else ""),
                           "instances_per_step": w.batch * w.heads,
                           "l2": "6.3 GB of Q, K, V per step exceed the 126 MB L2"},
                "clocks": clocks,
                "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": "head-tokens/s",
                        "h2d_bytes_per_step": (Q.numel() + Kp.numel() + V.numel()) * 2, "d2h_bytes_per_step": rec_bytes},
                "gpu_launches": int(launches),
                "roofline": {"bound": "tensor", "kernel": {"build": "state_tc_kernel"}.get(dominant, dominant + "_tc_kernel"), "achieved": ach, "peak": peak,
                             "unit": "TFLOP/s", "frac": ach / peak, "peak_kind": kind, "traffic": None,
                             "algorithmic_flops_per_launch": fl[dominant],
                             "kernel_ms": {k: v for k, v in kt.items() if v},
                             "kernel_TFLOPs": {k: fl[k] / (kt[k] * 1e-3) / 1e12 for k in fl if kt.get(k)}}}
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()

def run_masked(args):
    """The parallel form: a step = less_masked_attention over one layer (B x heads sequences)."""
    import torch
    import torch.distributed as dist
    from paper_2402_09398_b200 import binding, build, workloads as wl
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the LESS path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
    build.build()
    S = args.seq
    w = wl.CONFIGS[2].with_(batch=args.batch or 2, prompt=S, heavy=int(0.05 * S), recent=int(0.05 * S))
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

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(W_steps):
        one_step()
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ctx.launches
    t0 = time.time()
    e0.record(stream)
    for _ in range(K_steps):
        one_step()
    e1.record(stream)
    barrier()
    t1 = time.time()
    launches = ctx.launches - launches0
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop(t0, t1) if sampler else None
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
    if ctx.poll_status() != 0:
        raise RuntimeError("device status")
    ms, ms_e2e = max_over_ranks([ms, ms_e2e], dev, world)
    if rank == 0:
        inst = w.batch * w.heads
        tokens = inst * S * world
        causal = S * (S + 1) // 2
        # flops of the entries the kernel has to form: 128 x 128 tiles that are not dead (a key tile all of
        # whose keys were discarded before a Q tile's first row is handled through its summed state)
        nt = (S + 127) // 128
        eu_pad = torch.full((w.batch, 1, w.heads, nt * 128), 0, dtype=torch.int64, device=dev)
        eu_pad[..., :S] = eu.long()
        death = eu_pad.view(w.batch, 1, w.heads, nt, 128).amax(-1)
        first_dead = torch.maximum((death + 127) // 128, torch.arange(nt, device=dev) + 1).clamp(max=nt)
        live_pairs = int((first_dead - torch.arange(nt, device=dev)).sum().item())
        live_frac = live_pairs / (inst * nt * (nt + 1) / 2)
        fl = {"masked_out": live_pairs * 128 * 128 * (4 * w.head_dim + 2 * w.rank),
              "psi": inst * S * 2 * (2 * w.head_dim * w.hidden + 2 * w.hidden * w.rank + w.rank * w.rank)}
        kt = {k: (prof[k][0] / prof[k][1] if prof[k][1] else 0.0) for k in prof}
        kt["psi"] *= 2                                   # psi and phi launches are booked under the same id
        kt["masked_pack"] *= 3                           # operand pack, tile states, running sums
        dominant = max(fl, key=lambda k: kt.get(k, 0.0))
        pth = os.path.join(ROOT, "MEASURED_PEAKS.json")
        peak, kind = (float(json.load(open(pth))["bf16_tflops_sustained"]), "of measured (sustained bf16 = fp16 rate)") \
            if os.path.exists(pth) else (1400.0, "of fallback")
        ach = fl[dominant] / (kt[dominant] * 1e-3) / 1e12 if kt.get(dominant) else 0.0
        line = {"metric": "parallel-form head-tokens/s (one layer per step)", "value": tokens * K_steps / (ms * 1e-3),
                "unit": "head-tokens/s", "n_gpus": world, "steps": K_steps, "warmup": W_steps, "ms_per_step": ms / K_steps,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "f16 inputs, f32 accumulate", "data": "synthetic",
                "config": {"workload": f"parallel form (B={w.batch}, {w.heads} heads, sequences of {S}, one layer per step, R={w.rank})",
                           "instances_per_step": inst, "live_tile_fraction": live_frac, "l2": "inputs, operands and output of a step exceed the 126 MB L2"
                           if inst * S * 1300 > 126e6 else "a step's data fit the L2"},
                "clocks": clocks,
                "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": "head-tokens/s",
                        "h2d_bytes_per_step": 3 * Q.numel() * 2 + eu.numel() * 4, "d2h_bytes_per_step": out.numel() * 4},
                "gpu_launches": int(launches),
                "roofline": {"bound": "tensor", "kernel": "masked_out_tc_kernel" if dominant == "masked_out" else dominant,
                             "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak, "peak_kind": kind,
                             "traffic": None, "algorithmic_flops_per_launch": fl[dominant],
                             "kernel_ms": {k: v for k, v in kt.items() if v}}}
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.masked_form:
        if args.steps == 1000:
            args.steps = 20
        run_masked(args)
    elif args.config == 5:
        if args.steps == 1000:
            args.steps = 5                # a step here is ~0.1 s of tensor-core work, not ~0.1 ms
        run_prefill(args)
    else:
        run_b200(args)


if __name__ == "__main__":
    main()
