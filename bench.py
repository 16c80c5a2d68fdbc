#!/usr/bin/env python
"""Benchmark of the MoE-layer decode step (spice_moe_layer_fwd) on B200.

One step = one pass of the whole hot path (route, classify, grouped expert FFN over the
resident slots, shared expert + LoRE surrogate, combine) over one decode batch of a
DeepSeek-V2-Lite-shaped layer.  Successive steps rotate through several independent
layer weight sets so that the bytes touched between two uses of the same weights are
several times the L2 capacity (cold-L2 timing without a flush inside the timed region).
Decode steps are submitted as replayed CUDA graphs of captured steps (--launch eager: one call per step); batches above
64 tokens, a dozen kernels on two streams per step, as one library call per step.

Prints ONE JSON line: metric, value, unit, timing, `config` (the workload), `roofline` (algorithmic bytes or FLOPs of
the timed calls over their time, against the measured peak), `e2e` (the same metric with host<->device copies inside
the timed region), `cpu_baseline` (the CPU oracle on the host cores), `clocks`, `gpu_launches`.

Other modes: --stack (26-layer decode stack), --op draft_confidence, --op rollout, --impl reference (CPU oracle).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "moe_layer_decode_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu captures summarised under
# profiles/ (same workload with 2 weight sets; mean of the two captured launches), keyed by (shape, tokens, path)
CAPTURED_TRAFFIC = {("dsv2lite", 16, 0, "bf16"): (502.9e6, "profiles/decode_tc_kernel_dsv2lite_T16.md"),
                    ("dsv2lite", 16, 0, "fp8"): (259.1e6, "profiles/decode_tc_kernel_fp8.md")}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            with open(p) as f:
                d = json.load(f)
            return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]), "source": "measured"}
        except Exception:
            pass
    return {**FALLBACK_PEAKS, "source": "fallback"}


# ----------------------------------------------------------------------------- clocks sampler
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.samples = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={gpu_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 6:
                try:
                    self.samples.append((time.time(), float(parts[0]), float(parts[1]), parts[2:6]))
                except ValueError:
                    pass

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()

    def summary(self, t0: float, t1: float):
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        win = [s for s in self.samples if t0 <= s[0] <= t1]
        where = "timed region"
        if not win:
            win = self.samples[-5:]
            where = "nearest samples (timed region shorter than the sampling period)"
        if not win:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "window": "none"}
        reasons = sorted({n for s in win for n, v in zip(names, s[3]) if v.lower().startswith("active")})
        return {"sm_mhz": float(np.median([s[1] for s in win])), "sm_max_mhz": float(max(s[2] for s in win)),
                "reasons": reasons, "samples": len(win), "window": where}


# ----------------------------------------------------------------------------- multi-rank plumbing
def max_over_ranks(values, device=None):
    """Element-wise maximum of per-rank timings (the slowest rank defines a step); identity for one rank."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_throughput(units_per_rank_per_step, steps, world, ms_max):
    """Replicas only: every rank runs the same number of units; the job's rate is all ranks' units over the slowest rank's time."""
    return world * units_per_rank_per_step * steps / (ms_max * 1e-3)


# ----------------------------------------------------------------------------- workload
def algorithmic_bytes(shape, T, idx, cls, fp8=False):
    """Bytes the method must move for one layer call (weights read once per distinct expert: bf16, or for fp8 one byte
    per expert weight plus a 4-byte scale per weight row; router and LoRE factors are bf16 in both)."""
    s = shape
    hit = {int(e) for e, c in zip(idx.ravel(), cls.ravel()) if c == 0}
    low = {int(e) for e, c in zip(idx.ravel(), cls.ravel()) if c == 2}
    expert_w = 3 * s.d * s.inter_shared + len(hit) * 3 * s.d * s.inter
    if fp8:
        expert_w = expert_w + 4 * ((2 * s.inter_shared + s.d) + len(hit) * (2 * s.inter + s.d))
    else:
        expert_w = 2 * expert_w
    w = 2 * (s.n_experts * s.d + len(low) * 2 * s.lore_rank * s.d) + expert_w
    act = 2 * T * s.d + 2 * T * s.d + 4 * T * s.top_k
    return w + act, len(hit), len(low)


def device_replica(torch, B, shape, gen, dev):
    """A layer weight set drawn on the device: N(0, 0.02) bf16, random residency of S experts."""
    s = shape

    def rn(*sz):
        return (torch.randn(*sz, generator=gen, device=dev, dtype=torch.float32) * 0.02).to(torch.bfloat16)

    gu = torch.empty(s.n_slots, 2 * s.inter, s.d, dtype=torch.bfloat16, device=dev)
    dn = torch.empty(s.n_slots, s.d, s.inter, dtype=torch.bfloat16, device=dev)
    for i in range(s.n_slots):
        gu[i] = rn(2 * s.inter, s.d)
        dn[i] = rn(s.d, s.inter)
    perm = torch.randperm(s.n_experts, generator=gen, device=dev)
    soe = torch.full((s.n_experts,), -1, dtype=torch.int32, device=dev)
    soe[perm[: s.n_slots]] = torch.arange(s.n_slots, dtype=torch.int32, device=dev)
    return B.LayerWeights(w_router=rn(s.n_experts, s.d), slot_w_gate_up=gu, slot_w_down=dn, slot_of_expert=soe,
                          shared_w_gate_up=rn(2 * s.inter_shared, s.d), shared_w_down=rn(s.d, s.inter_shared),
                          lore_A=rn(s.n_experts, s.lore_rank, s.d), lore_B=rn(s.n_experts, s.d, s.lore_rank))


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2608_21240_b200 import binding as B
    from paper_2608_21240_b200 import workloads as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    B.lib()   # fail loudly when the extension is missing

    shape = W.SHAPES[args.shape]
    T, R = args.tokens, args.replicas
    peaks = load_peaks()

    # replica 0 comes from the numpy generator (the CPU baseline needs the same numbers);
    # the others are drawn on the device with the same distributions
    prefill = T > 64   # large batch: the grouped GEMM is tensor-bound; use the skewed (Zipf) router of config 4
    zipf = prefill if args.router == "auto" else args.router == "zipf"
    wl0 = W.make_layer(shape, T, variant=100 + rank, zipf=zipf)
    upload, bf16_tensor, cfg_of = B.upload, B.bf16_tensor, B.cfg_of
    gen = torch.Generator(device=dev)
    gen.manual_seed(W.BASE_SEED + 1000 * rank)
    reps = [upload(wl0, dev)] + [device_replica(torch, B, shape, gen, dev) for _ in range(R - 1)]
    if zipf:
        for r in reps[1:]:
            r.w_router.copy_(reps[0].w_router)   # same popularity skew in every weight set
    fp8 = args.dtype == "fp8"
    if fp8:
        reps = [B.quantize_layer(r) for r in reps]      # the bf16 sets are released once quantised
        torch.cuda.synchronize()
    structs = [r.c_struct() for r in reps]
    layer_call = B.spice_moe_layer_fwd_fp8 if fp8 else B.spice_moe_layer_fwd
    h = bf16_tensor(wl0.h, dev)
    conf = torch.from_numpy(wl0.conf).to(dev)
    layer = B.SpiceLayer(cfg_of(shape), T, device=local)
    if args.path:
        layer.set_option(B.OPT_PATH, args.path)
    y = torch.empty(T, shape.d, dtype=torch.bfloat16, device=dev)
    idx = torch.empty(T, shape.top_k, dtype=torch.int32, device=dev)
    gate = torch.empty(T, shape.top_k, dtype=torch.float32, device=dev)
    cls = torch.empty(T, shape.top_k, dtype=torch.uint8, device=dev)
    counts = torch.zeros(3, dtype=torch.int32, device=dev)
    # residual-miss list (set M of Sec. 4.3): part of the call's output, written in the timed region
    n_ent = T * shape.top_k
    resid = (torch.empty(n_ent, dtype=torch.int32, device=dev), torch.empty(n_ent, dtype=torch.int32, device=dev),
             torch.empty(n_ent, dtype=torch.int32, device=dev), torch.empty(n_ent, dtype=torch.float32, device=dev))
    stream = torch.cuda.current_stream()

    def step(i):
        layer_call(layer.ctx, structs[i % R], h, conf, T, y, idx=idx, gate=gate, cls=cls, counts=counts,
                              resid_tok=resid[0], resid_k=resid[1], resid_expert=resid[2], resid_gate=resid[3],
                              stream=torch.cuda.current_stream())

    # algorithmic bytes of every replica's call (from the routing the library itself produced)
    rep_bytes, rep_hit, rep_low, rep_hit_picks = [], [], [], []
    for i in range(R):
        step(i)
        torch.cuda.synchronize()
        b, nh, nl = algorithmic_bytes(shape, T, idx.cpu().numpy(), cls.cpu().numpy(), fp8)
        rep_bytes.append(b)
        rep_hit.append(nh)
        rep_low.append(nl)
        rep_hit_picks.append(float((cls.cpu().numpy() == 0).sum()) / T)   # exact expert evaluations per token

    sampler = ClockSampler(local) if rank == 0 else None
    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    l0 = layer.launch_count()
    step(0)
    launches_per_step = layer.launch_count() - l0
    launch = args.launch if args.launch != "auto" else ("eager" if prefill else "graph")
    ms, how, w0, w1 = timed_steps(torch, step, args.steps, launch)
    if world > 1:
        dist.barrier()
    launches = launches_per_step * args.steps
    total_bytes = sum(rep_bytes[i % R] for i in range(args.steps))

    # end to end: inputs start in pinned host memory, the result is read back to the host every step.  The caller
    # packs what travels together: one pinned block (h, conf) -> one device block, one device block (y, counts) -> host.
    in_bytes = h.numel() * 2 + conf.numel() * 4
    in_host = torch.empty(in_bytes, dtype=torch.uint8).pin_memory()
    in_dev = torch.empty(in_bytes, dtype=torch.uint8, device=dev)
    in_host[: h.numel() * 2].copy_(h.cpu().view(torch.uint8).reshape(-1))
    in_host[h.numel() * 2:].copy_(conf.cpu().view(torch.uint8).reshape(-1))
    h_dev = in_dev[: h.numel() * 2].view(torch.bfloat16).view(T, shape.d)
    conf_dev = in_dev[h.numel() * 2:].view(torch.float32).view_as(conf)
    # one device block -> host: y, the class counts, and the residual-miss list (the host runtime needs it to recover
    # those experts; its capacity T*K is copied, counts[1] entries of it are valid)
    y_bytes = T * shape.d * 2
    out_bytes = y_bytes + 16 + 16 * n_ent
    out_dev = torch.empty(out_bytes, dtype=torch.uint8, device=dev)
    out_host = torch.empty(out_bytes, dtype=torch.uint8).pin_memory()
    y_e2e = out_dev[:y_bytes].view(torch.bfloat16).view(T, shape.d)
    cnt_e2e = out_dev[y_bytes:y_bytes + 16].view(torch.int32)[:3]
    r0 = y_bytes + 16
    resid_e2e = tuple(out_dev[r0 + 4 * n_ent * j: r0 + 4 * n_ent * (j + 1)].view(torch.float32 if j == 3 else torch.int32)
                      for j in range(4))

    # --e2e-out copy (default): results are written to device memory and copied back as one block.
    # --e2e-out mapped: the call is given the pinned host block itself (device-accessible under unified addressing), so
    # the kernel's own stores carry y, the counts and the residual-miss list to the host and no copy-back node is needed.
    mapped = args.e2e_out == "mapped"
    if mapped:
        y_e2e = out_host[:y_bytes].view(torch.bfloat16).view(T, shape.d)
        cnt_e2e = out_host[y_bytes:y_bytes + 16].view(torch.int32)[:3]
        resid_e2e = tuple(out_host[r0 + 4 * n_ent * j: r0 + 4 * n_ent * (j + 1)].view(torch.float32 if j == 3 else torch.int32)
                          for j in range(4))

    def e2e_enqueue(i):
        st = torch.cuda.current_stream()
        in_dev.copy_(in_host, non_blocking=True)
        layer_call(layer.ctx, structs[i % R], h_dev, conf_dev, T, y_e2e, idx=idx, gate=gate, cls=cls,
                              counts=cnt_e2e, resid_tok=resid_e2e[0], resid_k=resid_e2e[1], resid_expert=resid_e2e[2],
                              resid_gate=resid_e2e[3], stream=st)
        if not mapped:
            out_host.copy_(out_dev, non_blocking=True)

    # a decode step (copy in, one kernel, copy out) is captured once per weight set and replayed; the host still
    # waits for every step's result before it submits the next one
    e2e_graphs = None
    if launch == "graph":
        try:
            e2e_graphs = []
            for i in range(R):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, capture_error_mode="thread_local"):
                    e2e_enqueue(i)
                e2e_graphs.append(g)
        except Exception:
            e2e_graphs = None

    def e2e_step(i):
        if e2e_graphs is not None:
            e2e_graphs[i % R].replay()
        else:
            e2e_enqueue(i)
        stream.synchronize()     # the caller consumes y before the next step

    for i in range(min(args.warmup, 5)):
        e2e_step(i)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    n_e2e = args.steps
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(stream)
    for i in range(n_e2e):
        e2e_step(i)
    f1.record(stream)
    torch.cuda.synchronize()
    w2 = time.time()
    ms_e2e = f0.elapsed_time(f1)
    if sampler:
        sampler.stop()
    # what reached the host in the last end-to-end step is what the device-resident call gives for that weight set
    step((n_e2e - 1) % R)
    torch.cuda.synchronize()
    got = out_host[:y_bytes].view(torch.bfloat16).view(T, shape.d)
    if not torch.equal(got, y.cpu()) or out_host[y_bytes:y_bytes + 12].view(torch.int32).tolist() != counts.cpu().tolist():
        raise SystemExit("end-to-end leg: the results in host memory differ from the device-resident call's")

    ms, ms_e2e = max_over_ranks([ms, ms_e2e], dev)
    status = layer.device_status()
    if status != 0:
        raise SystemExit(f"device status {status} after the timed region")

    if rank == 0:
        tok_s = whole_job_throughput(T, args.steps, world, ms)
        achieved = total_bytes / (ms * 1e-3) / 1e9
        if prefill:
            # tensor-bound: algorithmic FLOPs of the exact experts + shared expert (2 per multiply-add)
            flops = args.steps * T * 6.0 * shape.d * (float(np.mean(rep_hit_picks)) * shape.inter + shape.inter_shared)
            tfs = flops / (ms * 1e-3) / 1e12
        out = {
            "metric": METRIC, "value": tok_s, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "fp8_e4m3_weights_bf16_activations" if fp8 else "bf16", "data": "synthetic",
            "config": {"workload": f"{shape.name} decode layer, batch {T} tokens "
                                   f"(d={shape.d}, N={shape.n_experts}, K={shape.top_k}, I={shape.inter}, "
                                   f"I_s={shape.inter_shared}, r={shape.lore_rank}, {shape.n_slots} resident slots, "
                                   f"tau={shape.tau}, Beta(2,2) confidences)",
                       "weights": ("expert and shared-expert matrices as E4M3 bytes with one power-of-two scale per row "
                                   "(quantised on the device from the bf16 sets); router and LoRE factors bf16") if fp8 else "bf16",
                       "tokens_per_step": T, "cold_l2": f"steps rotate through {R} independent weight sets "
                       f"({sum(rep_bytes) / 1e6:.0f} MB between reuses, L2 is 126 MB); no flush in the timed region",
                       "launch": how,
                       "distinct_hit_experts_mean": float(np.mean(rep_hit)),
                       "distinct_lowconf_experts_mean": float(np.mean(rep_low)),
                       "multi_gpu": "replicas only (no collective on the data path)"},
            "roofline": ({"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                          "frac": achieved / peaks["hbm_gbs"],
                          "traffic": CAPTURED_TRAFFIC.get((shape.name, T, args.path, args.dtype), (None, None))[0],
                          "traffic_source": CAPTURED_TRAFFIC.get((shape.name, T, args.path, args.dtype), (None, None))[1],
                          "kernel": "all launches of spice_moe_layer_fwd (algorithmic bytes of the call / time per call)",
                          "algorithmic_bytes_per_step": total_bytes / args.steps, "peak_source": peaks["source"],
                          "frac_of_nominal_8TBs": achieved / 8000.0} if not prefill else
                         {"bound": "tensor", "achieved": tfs, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                          "frac": tfs / peaks["bf16_tflops"], "traffic": None,
                          "kernel": "whole spice_moe_layer_fwd call (expert + shared-expert FLOPs / time per call; "
                                    "the grouped GEMM kernels alone are in profiles/)",
                          "peak_source": peaks["source"], "frac_of_nominal_2250": tfs / 2250.0}),
            "e2e": {"value": whole_job_throughput(T, n_e2e, world, ms_e2e), "unit": UNIT,
                    "h2d_bytes_per_step": int(in_bytes), "d2h_bytes_per_step": int(out_bytes),
                    "ms_per_step": ms_e2e / n_e2e,
                    "launch": ("one replayed graph (copy in, call, copy out) and one stream synchronisation per step"
                               if e2e_graphs is not None else "copy in, library call, copy out, stream synchronisation per step"),
                    "results": "written by the kernel into pinned host memory (no copy-back node)" if mapped
                               else "one device block copied back"},
            "gpu_launches": int(launches),
            "clocks": sampler.summary(w0, w1) if sampler else None,
        }
        if not args.no_cpu_baseline and world == 1:
            out["cpu_baseline"] = cpu_baseline(wl0, budget_s=args.cpu_budget)
            out["cpu_baseline"]["one_thread"] = cpu_baseline_one_thread(args, 100 + rank, min(args.cpu_budget, 10.0))
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def timed_steps(torch, step_fn, n_steps, launch):
    """Times exactly n_steps calls of step_fn(i) (which enqueues step i on torch's current stream) with CUDA events.
    launch == "graph": the steps are captured into CUDA graphs of up to 256 steps and replayed, the way a decode loop
    submits a fixed layer call; launch == "eager": one library call per step from Python.  Returns (ms, description)."""
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    how = "one library call per step"
    plan = None
    if launch == "graph":
        try:
            chunk = min(n_steps, 256)
            sizes = [chunk] + ([n_steps % chunk] if n_steps % chunk else [])
            graphs = []
            for n in sizes:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, capture_error_mode="thread_local"):   # other threads (NCCL watchdog) may call CUDA
                    for i in range(n):
                        step_fn(i)
                graphs.append(g)
            plan = [graphs[0]] * (n_steps // chunk) + (graphs[1:] if n_steps % chunk else [])
            for g in graphs:
                g.replay()          # untimed: instantiates and uploads the graph
            how = f"CUDA graphs of {chunk} captured steps, replayed"
        except Exception as ex:     # capture refused: time the eager loop and say so
            plan = None
            how = f"one library call per step (graph capture failed: {type(ex).__name__})"
    torch.cuda.synchronize()
    w0 = time.time()
    e0.record(stream)
    if plan is not None:
        for g in plan:
            g.replay()
    else:
        for i in range(n_steps):
            step_fn(i)
    e1.record(stream)
    torch.cuda.synchronize()
    w1 = time.time()
    return e0.elapsed_time(e1), how, w0, w1


# ----------------------------------------------------------------------------- 26-layer decode stack (config 5)
def stack_residency(idx, n_experts, n_slots, tau, rng, hit_rate=0.7):
    """Residency and confidences of one layer GIVEN its routing (host logic of the input recipe, no method arithmetic):
    selected experts are made resident in random order until >= hit_rate of the picks hit, the remaining slots hold
    unselected experts (stale prefetches); a miss is low-confidence with probability 1/2."""
    picks = idx.ravel()
    selected = rng.permutation(np.unique(picks))
    resident, hits = [], 0
    for e in selected:
        if hits >= hit_rate * picks.size or len(resident) >= n_slots:
            break
        resident.append(int(e))
        hits += int((picks == e).sum())
    sel = set(selected.tolist())
    resident += [int(e) for e in rng.permutation(n_experts) if e not in sel][: n_slots - len(resident)]
    soe = np.full(n_experts, -1, np.int32)
    soe[np.array(resident)] = rng.permutation(len(resident)).astype(np.int32)
    conf = rng.random((idx.shape[0], n_experts)).astype(np.float32)
    for t in range(idx.shape[0]):
        for e in idx[t]:
            if soe[e] < 0:
                conf[t, e] = np.float32(rng.uniform(0.0, tau * 0.999) if rng.random() < 0.5 else rng.uniform(tau * 1.001, 1.0))
    return soe, conf


def run_stack(args):
    """--stack: one step = the MoE layers of a 26-layer DeepSeek-V2-Lite-shaped decoder for one decode batch of 8
    tokens, free running: 26 layer calls back to back on one stream, each with its own weights (13.5 GB in all, so
    the L2 is cold for every layer), the residual stream updated inside the call (x += y)."""
    import torch
    import torch.distributed as dist

    from paper_2608_21240_b200 import binding as B
    from paper_2608_21240_b200 import workloads as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    B.lib()
    shape = W.SHAPES["dsv2lite_stack"]
    T, n_layers = 8, 26
    peaks = load_peaks()
    gen = torch.Generator(device=dev)
    gen.manual_seed(W.BASE_SEED + 5000 + 1000 * rank)
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([W.BASE_SEED, 5, 777, rank])))
    layer = B.SpiceLayer(B.cfg_of(shape), T, device=local)
    if args.path:
        layer.set_option(B.OPT_PATH, args.path)
    stream = torch.cuda.current_stream()
    weights, hs, confs = [], [], []
    idx = torch.empty(T, shape.top_k, dtype=torch.int32, device=dev)
    gate = torch.empty(T, shape.top_k, dtype=torch.float32, device=dev)
    cls = torch.empty(T, shape.top_k, dtype=torch.uint8, device=dev)
    for l in range(n_layers):
        w = device_replica(torch, B, shape, gen, dev)
        h = torch.randn(T, shape.d, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
        B.spice_route_topk(layer.ctx, h, w.w_router, T, idx, gate, stream=stream)
        torch.cuda.synchronize()
        soe, conf = stack_residency(idx.cpu().numpy(), shape.n_experts, shape.n_slots, shape.tau, rng)
        w.slot_of_expert.copy_(torch.from_numpy(soe))
        weights.append(w)
        hs.append(h)
        confs.append(torch.from_numpy(conf).to(dev))
    structs = [w.c_struct() for w in weights]
    x = torch.zeros(T, shape.d, dtype=torch.bfloat16, device=dev)      # residual stream
    y = torch.empty(T, shape.d, dtype=torch.bfloat16, device=dev)

    def step():
        for l in range(n_layers):
            B.spice_moe_layer_fwd(layer.ctx, structs[l], hs[l], confs[l], T, y, x_resid=x, idx=idx, cls=cls,
                                  stream=torch.cuda.current_stream())

    total_bytes, hit_frac = 0, []
    for l in range(n_layers):
        B.spice_moe_layer_fwd(layer.ctx, structs[l], hs[l], confs[l], T, y, idx=idx, cls=cls, stream=stream)
        torch.cuda.synchronize()
        b, _, _ = algorithmic_bytes(shape, T, idx.cpu().numpy(), cls.cpu().numpy())
        total_bytes += b
        hit_frac.append(float((cls.cpu().numpy() == 0).mean()))
    sampler = ClockSampler(local) if rank == 0 else None
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    l0 = layer.launch_count()
    step()
    launches_per_step = layer.launch_count() - l0
    ms, how, w0, w1 = timed_steps(torch, lambda i: step(), args.steps, "eager" if args.launch == "eager" else "graph")
    if world > 1:
        dist.barrier()
    launches = launches_per_step * args.steps
    # end to end: the residual stream comes from pinned host memory and goes back every step
    x_host = torch.zeros(T, shape.d, dtype=torch.bfloat16).pin_memory()
    out_host = torch.empty(T, shape.d, dtype=torch.bfloat16).pin_memory()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_e2e = args.steps
    f0.record(stream)
    for _ in range(n_e2e):
        x.copy_(x_host, non_blocking=True)
        step()
        out_host.copy_(x, non_blocking=True)
        stream.synchronize()
    f1.record(stream)
    torch.cuda.synchronize()
    ms_e2e = f0.elapsed_time(f1)
    if sampler:
        sampler.stop()
    ms, ms_e2e = max_over_ranks([ms, ms_e2e], dev)
    status = layer.device_status()
    if status != 0:
        raise SystemExit(f"device status {status} after the timed region")
    if rank == 0:
        achieved = total_bytes * args.steps / (ms * 1e-3) / 1e9
        out = {
            "metric": "moe_stack_decode_tokens_per_s", "value": whole_job_throughput(T, args.steps, world, ms), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"MoE layers of a {n_layers}-layer DeepSeek-V2-Lite-shaped decoder, decode batch {T}, "
                                   f"free running ({shape.n_slots} resident slots per layer, residency chosen given the "
                                   f"routing: mean hit rate {np.mean(hit_frac):.2f}, misses low-confidence w.p. 1/2)",
                       "tokens_per_step": T, "layer_calls_per_step": n_layers, "launch": how,
                       "cold_l2": f"every layer has its own weights ({total_bytes / 1e6:.0f} MB touched per step, "
                                  f"L2 is 126 MB); no flush in the timed region",
                       "multi_gpu": "replicas only (no collective on the data path)"},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": achieved / peaks["hbm_gbs"], "traffic": None,
                         "kernel": "all 26 launches of a step (sum of the calls' algorithmic bytes / time per step)",
                         "algorithmic_bytes_per_step": float(total_bytes), "peak_source": peaks["source"]},
            "e2e": {"value": whole_job_throughput(T, n_e2e, world, ms_e2e), "unit": UNIT,
                    "h2d_bytes_per_step": int(x_host.numel() * 2), "d2h_bytes_per_step": int(out_host.numel() * 2),
                    "ms_per_step": ms_e2e / n_e2e},
            "gpu_launches": int(launches),
            "clocks": sampler.summary(w0, w1) if sampler else None,
            "cpu_baseline": None,
        }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- draft-router confidence (Sec. 4.1)
def run_draft_confidence(args):
    """--op draft_confidence: one step = spice_draft_confidence over one batch (router copy of one layer)."""
    import torch

    from paper_2608_21240_b200 import binding as B
    from paper_2608_21240_b200 import workloads as W
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    B.lib()
    shape = W.SHAPES[args.shape]
    T, R = args.tokens, max(args.replicas, 64)
    gen = torch.Generator(device=dev)
    gen.manual_seed(W.BASE_SEED + 77)
    routers = [(torch.randn(shape.n_experts, shape.d, generator=gen, device=dev) * 0.02).to(torch.bfloat16) for _ in range(R)]
    hs = [torch.randn(T, shape.d, generator=gen, device=dev).to(torch.bfloat16) for _ in range(R)]
    layer = B.SpiceLayer(B.cfg_of(shape), T, device=dev.index)
    idx = torch.empty(T, shape.top_k, dtype=torch.int32, device=dev)
    conf = torch.empty(T, dtype=torch.float32, device=dev)
    pi = torch.empty(T, shape.n_experts, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def step(i):
        B.spice_draft_confidence(layer.ctx, hs[i % R], routers[i % R], T, idx, conf, pi, stream=stream)

    for i in range(args.warmup):
        step(i)
    flush.fill_(1)        # cold L2 at the start; the rotating inputs (R sets) keep the router rows out of L1
    torch.cuda.synchronize()
    l0 = layer.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    nbytes = 2 * shape.n_experts * shape.d + 2 * T * shape.d + 4 * T * (shape.n_experts + shape.top_k + 1)
    peaks = load_peaks()
    achieved = nbytes * args.steps / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": "draft_confidence_tokens_per_s", "value": T * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"draft-router confidence, {shape.name} router (N={shape.n_experts}, d={shape.d}, K={shape.top_k}), "
                               f"batch {T} tokens, {R} rotating input sets (warm L2: {R * nbytes / 1e6:.1f} MB in all)"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved / peaks["hbm_gbs"], "traffic": None,
                     "kernel": "route_topk_kernel + draft_confidence_kernel (latency-bound at decode batches: "
                               "the call moves well under a megabyte)", "peak_source": peaks["source"]},
        "gpu_launches": int(layer.launch_count() - l0)}))


# ----------------------------------------------------------------------------- Algorithm 1 rollout
def run_rollout(args):
    """--op rollout: one step = spice_prefetch_rollout (Algorithm 1) over one decode batch, l_min = 2, l_max = 4."""
    import torch

    from paper_2608_21240_b200 import binding as B
    from paper_2608_21240_b200 import workloads as W
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    B.lib()
    shape = W.SHAPES[args.shape]
    T, l_min, l_max = args.tokens, 2, 4
    R = max(2, min(args.replicas, 8))          # rotating sets of l_max layers
    gen = torch.Generator(device=dev)
    gen.manual_seed(W.BASE_SEED + 99)

    def rn(*sz):
        return (torch.randn(*sz, generator=gen, device=dev, dtype=torch.float32) * 0.02).to(torch.bfloat16)

    s = shape
    dummy = torch.zeros(8, dtype=torch.bfloat16, device=dev)
    soe = torch.full((s.n_experts,), -1, dtype=torch.int32, device=dev)
    sets = [[B.LayerWeights(w_router=rn(s.n_experts, s.d), slot_w_gate_up=dummy, slot_w_down=dummy, slot_of_expert=soe,
                            shared_w_gate_up=rn(2 * s.inter_shared, s.d), shared_w_down=rn(s.d, s.inter_shared),
                            lore_A=rn(s.n_experts, s.lore_rank, s.d), lore_B=rn(s.n_experts, s.d, s.lore_rank))
             for _ in range(l_max)] for _ in range(R)]
    structs = [[w.c_struct() for w in ws] for ws in sets]
    x = torch.randn(T, s.d, generator=gen, device=dev).to(torch.bfloat16)
    layer = B.SpiceLayer(B.cfg_of(shape), T, device=dev.index)
    idx = torch.empty(l_max, T, s.top_k, dtype=torch.int32, device=dev)
    conf = torch.empty(l_max, T, dtype=torch.float32, device=dev)
    depth = torch.empty(T, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    # a threshold that stops about half of the tokens at l_min: the median confidence at that depth
    B.spice_prefetch_rollout(layer.ctx, structs[0], x, T, l_min, l_max, 0.0, idx, conf, depth, stream=stream)
    torch.cuda.synchronize()
    tau = float(conf[l_min - 1].median().item())

    def step(i):
        B.spice_prefetch_rollout(layer.ctx, structs[i % R], x, T, l_min, l_max, tau, idx, conf, depth, stream=stream)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    l0 = layer.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    mean_depth = float(depth.float().mean().item())
    nbytes = (l_max - 1) * 2 * (s.n_experts * s.d + 3 * s.d * s.inter_shared) + 2 * s.n_experts * s.d
    peaks = load_peaks()
    achieved = nbytes * args.steps / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": "prefetch_rollout_tokens_per_s", "value": T * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"Algorithm 1 rollout, {shape.name}-shaped layers (router, shared expert, LoRE factors), batch {T} "
                               f"tokens, l_min={l_min}, l_max={l_max}, tau={tau:.3f} (median confidence at l_min), mean depth "
                               f"{mean_depth:.2f}, {R} rotating sets of {l_max} layers"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved / peaks["hbm_gbs"], "traffic": None,
                     "kernel": "all launches of the call; bytes = routers and shared experts of the depths that project "
                               "(LoRE factors of the selected experts not counted)", "peak_source": peaks["source"]},
        "gpu_launches": int(layer.launch_count() - l0)}))


# ----------------------------------------------------------------------------- LoRE calibration
def run_lore_calibrate(args):
    """--op lore_calibrate: one step = spice_lore_calibrate for one expert (n calibration tokens, 100 iterations)."""
    import torch

    from paper_2608_21240_b200 import binding as B
    from paper_2608_21240_b200 import workloads as W
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    B.lib()
    shape = W.SHAPES[args.shape]
    d, r, n, iters = shape.d, shape.lore_rank, max(args.tokens, 2 * shape.d), 100
    gen = torch.Generator(device=dev)
    gen.manual_seed(W.BASE_SEED + 55)
    h = torch.randn(n, d, generator=gen, device=dev).to(torch.bfloat16)
    m = torch.randn(d, d, generator=gen, device=dev) * (0.97 ** torch.arange(d, device=dev))
    resid = (h.float() @ m.T + 0.1 * torch.randn(n, d, generator=gen, device=dev)).contiguous()
    steps = max(1, min(args.steps, 10))
    for _ in range(2):
        out = B.spice_lore_calibrate(h, resid, r, iterations=iters)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        A, Bm, loss, status = B.spice_lore_calibrate(h, resid, r, iterations=iters)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    dp, rp = (d + 63) // 64 * 64, (r + 63) // 64 * 64
    flops = 2.0 * (2 * n * dp * dp + dp ** 3 / 3 + dp ** 3 + iters * 2 * dp * dp * rp + 2 * dp * dp * rp)
    print(json.dumps({
        "metric": "lore_calibrations_per_s", "value": 1e3 / ms, "unit": "experts/s", "n_gpus": 1, "steps": steps, "warmup": 2,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"LoRE calibration of one expert, d={d}, rank={r}, {n} calibration tokens, {iters} subspace "
                               f"iterations; objective / sum resid^2 = {float(loss[0] / loss[1]):.4f}, status {int(status.item())}"},
        "roofline": {"bound": "alu", "achieved": flops / (ms * 1e-3) / 1e12, "peak": 72.0, "unit": "TFLOP/s",
                     "frac": flops / (ms * 1e-3) / 1e12 / 72.0, "traffic": None,
                     "kernel": "Gram and subspace-iteration products on the tensor cores, blocked Cholesky / triangular solves in "
                               "fp32 SIMT; a chain of ~1400 small dependent launches (offline path)",
                     "peak_source": "148 SMs x 128 fp32 FMA lanes x 1.9 GHz x 2"},
        "gpu_launches": None}))


# ----------------------------------------------------------------------------- CPU oracle legs
def oracle_call(wl, tokens):
    """One oracle evaluation of the GPU part of the layer for the given tokens."""
    import oracle
    from tests._cases import run_oracle
    return run_oracle(wl, tokens=tokens, want_full=False)


def cpu_baseline(wl, budget_s=15.0):
    """The oracle, as it stands, timed on this machine's host cores on a bounded sample of the same batch: the whole batch
    when one pass fits the budget (decode batches), else as many of its tokens as do (large batches)."""
    import oracle
    T = wl.T
    oracle_call(wl, [0])                      # draws the first token's experts
    t0 = time.time()
    oracle_call(wl, [0])
    t_one = time.time() - t0
    n_tok = int(max(1, min(T, 0.5 * budget_s / max(t_one, 1e-4))))
    toks = list(range(n_tok))
    oracle_call(wl, toks)                     # draws the needed expert weights, warms caches
    t0 = time.time()
    reps = 0
    while True:
        oracle_call(wl, toks)
        reps += 1
        if time.time() - t0 > budget_s or reps >= 20:
            break
    dt = (time.time() - t0) / reps
    sample = (f"the full batch of {T} tokens of weight set 0" if n_tok == T else
              f"{n_tok} of the batch's {T} tokens (weight set 0)") + f", {reps} repetitions, mean"
    return {"value": n_tok / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample,
            "s_per_step": dt}


def cpu_baseline_one_thread(args, variant, budget_s):
    """The same oracle leg on ONE host thread: a child process with OMP_NUM_THREADS=1 (the oracle's only parallelism is
    OpenMP over independent outputs) re-creates the workload from its seed and prints its cpu_baseline object."""
    env = dict(os.environ, OMP_NUM_THREADS="1")
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        env.pop(k, None)
    cmd = [sys.executable, os.path.abspath(__file__), "--cpu-leg", str(variant), "--shape", args.shape, "--tokens",
           str(args.tokens), "--cpu-budget", str(budget_s), "--router", args.router]
    try:
        r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=60 + 20 * budget_s)
        return json.loads(r.stdout.strip().splitlines()[-1])
    except Exception as ex:
        return {"unavailable": f"{type(ex).__name__}: {ex}"}


def run_cpu_leg(args):
    from paper_2608_21240_b200 import workloads as W
    shape = W.SHAPES[args.shape]
    zipf = (args.tokens > 64) if args.router == "auto" else args.router == "zipf"
    wl = W.make_layer(shape, args.tokens, variant=args.cpu_leg, zipf=zipf)
    print(json.dumps(cpu_baseline(wl, budget_s=args.cpu_budget)))


def run_reference(args):
    """--impl reference: the CPU oracle timed on the host cores (there is no reference implementation)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2608_21240_b200 import workloads as W
    shape = W.SHAPES[args.shape]
    T = args.tokens
    wl = W.make_layer(shape, T, variant=100)
    t0 = time.time()
    oracle_call(wl, [0])
    oracle_call(wl, list(range(T)))          # draw all needed experts once
    t0 = time.time()
    oracle_call(wl, [0])
    t_one = time.time() - t0
    budget = 150.0
    n_tok = int(max(1, min(T, budget / max(1e-3, (args.steps + args.warmup) * t_one))))
    toks = list(range(n_tok))
    for _ in range(args.warmup):
        oracle_call(wl, toks)
    t0 = time.time()
    for _ in range(args.steps):
        oracle_call(wl, toks)
    dt = time.time() - t0
    val = n_tok * args.steps / dt
    sample = f"{n_tok} of the batch's {T} tokens per step (weight set 0)"
    out = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": f"{shape.name} decode layer, batch {T} tokens (CPU oracle, {sample})"},
           "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
           "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--shape", default="dsv2lite")
    ap.add_argument("--tokens", type=int, default=16)
    ap.add_argument("--replicas", type=int, default=8)
    ap.add_argument("--path", type=int, default=0,
                    help="kernel path (SPICE_OPT_PATH): 0 auto, 1 general kernels, 2 no fused kernel, 3 mma.sync decode kernel")
    ap.add_argument("--stack", action="store_true",
                    help="time the MoE layers of the 26-layer stack at decode batch 8 (one step = 26 layer calls)")
    ap.add_argument("--op", default="layer", choices=["layer", "draft_confidence", "rollout", "lore_calibrate", "plumbing"],
                    help="what a step is: the MoE layer call (default) or the draft-router confidence call")
    ap.add_argument("--router", default="auto", choices=["auto", "uniform", "zipf"],
                    help="router of the synthetic layer: i.i.d. weights (uniform loads) or the Zipf-skewed one of config 4; "
                         "auto = uniform for decode batches, zipf above 64 tokens")
    ap.add_argument("--launch", default="auto", choices=["auto", "graph", "eager"],
                    help="how the timed steps are submitted: replayed CUDA graphs of captured steps, or one library call per "
                         "step; auto = graphs for decode batches (one kernel per step, launch-bound), calls for batches "
                         "above 64 tokens (a dozen kernels on two streams per step)")
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "fp8"],
                    help="weight precision of the expert matrices: bf16, or fp8 = E4M3 bytes with a scale per row "
                         "(spice_moe_layer_fwd_fp8; decode batches up to 32 tokens)")
    ap.add_argument("--e2e-out", default="mapped", choices=["copy", "mapped"],
                    help="end-to-end leg: copy the results back as one block, or let the kernel write them into pinned host memory")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--cpu-leg", type=int, default=None, help=argparse.SUPPRESS)   # child of cpu_baseline_one_thread
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.cpu_leg is not None:
        run_cpu_leg(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_ranks(args)      # no launcher around us: start the N ranks ourselves
        return
    if "WORLD_SIZE" in os.environ and int(os.environ["WORLD_SIZE"]) != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but the launcher started WORLD_SIZE={os.environ['WORLD_SIZE']} ranks")
    dispatch(args)


def dispatch(args):
    if args.impl == "reference":
        run_reference(args)
    elif args.op == "draft_confidence":
        run_draft_confidence(args)
    elif args.op == "rollout":
        run_rollout(args)
    elif args.op == "lore_calibrate":
        run_lore_calibrate(args)
    elif args.op == "plumbing":
        run_plumbing(args)
    elif args.stack:
        run_stack(args)
    else:
        run_ours(args)


def _rank_main(local_rank, args, port):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(local_rank), LOCAL_RANK=str(local_rank),
                      WORLD_SIZE=str(args.gpus))
    dispatch(args)


def spawn_ranks(args):
    """`python bench.py --gpus N` without a launcher: N processes on this node, one per GPU (rank = local rank = GPU
    index), rendezvous on 127.0.0.1.  The ranks are replicas: they meet only at barriers and for the max over the ranks'
    timings; rank 0 prints the JSON line."""
    import socket

    import torch.multiprocessing as mp
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    mp.spawn(_rank_main, args=(args, port), nprocs=args.gpus, join=True)


def run_plumbing(args):
    """--op plumbing: the multi-rank scaffolding alone (process group, barriers, max over ranks, whole-job rate, one JSON
    line from rank 0) around a stand-in step that only sleeps.  Needs no GPU (gloo on CPU); it exists so that the N > 1
    entry of this file can be exercised where there is one GPU or none."""
    import torch
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    t0 = time.time()
    for _ in range(args.steps):
        time.sleep(1e-3 * (1 + rank))        # rank r is (1 + r) ms per step: the slowest rank must define the time
    ms = (time.time() - t0) * 1e3
    if world > 1:
        dist.barrier()
    (ms_max,) = max_over_ranks([ms])
    if rank == 0:
        print(json.dumps({"metric": "plumbing_units_per_s", "value": whole_job_throughput(args.tokens, args.steps, world, ms_max),
                          "unit": "units/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                          "ms_per_step": ms_max / args.steps, "ms_rank0": ms / args.steps, "higher_is_better": True,
                          "scaling": "weak", "data": "none (sleep)", "gpu_launches": 0}))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
