#!/usr/bin/env python
"""Benchmark of the KV-chunk stitching path on B200.

A step is one pass of the whole path over one batch of synthetic requests:
    kvb_assemble_select (stitch + deviation sums in one kernel, then the selection) -> kvb_selective_attn
(`--path two-call`: kvb_assemble -> kvb_deviation_topk -> kvb_selective_attn, the same work in three calls)
Default workload (N=1): the Qwen2.5-3B-shaped 2048-token prompt (12 int8 chunks + 4 fresh), one
request per step, rotating through enough independent replicas that the working set is far
larger than L2.  `--workload cfg2|cfg4` selects the long int4 prompt (with its selective
attention) or the ragged 32-request batch.

  python bench.py --gpus N --steps K --warmup W [--workload cfg1] [--impl reference]

Prints one JSON line (rank 0).  `--impl reference` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_21362_b200 import synth  # noqa: E402

METRIC = "assembled KV tokens/s (whole path: stitch + deviation top-k + selective attention)"
UNIT = "tokens/s"
WORKLOADS = {"cfg1": 1, "cfg2": 2, "cfg4": 4}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_burst": d["bf16_tflops"], "bf16_sustained": d["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


# --------------------------------------------------------------------------------------- clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) every few ms."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop_evt = threading.Event()
        self.active = False
        self.error = None

    def run(self):
        try:
            import pynvml as nv

            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {
                "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            }
            get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons
            while not self._stop_evt.is_set():
                if self.active:
                    self.samples.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                    r = get_reasons(h)
                    for k, bit in names.items():
                        if r & bit:
                            self.reasons.add(k)
                time.sleep(0.002)
            nv.nvmlShutdown()
        except Exception as e:  # clocks are evidence, not a dependency
            self.error = repr(e)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0, "error": self.error}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


# --------------------------------------------------------------------------------------- replicas
class Replica:
    """One independent copy of the workload's requests on the device, with its marshalled tables."""

    def __init__(self, B, ctx, wl, dev, seed_shift, meta_fp16=False):
        wl = synth.Workload(wl.name, wl.seed + 7919 * seed_shift, wl.shape, wl.requests, wl.select, wl.sigma_bulk, wl.sigma_seam, wl.seam_tokens)
        qk, qv = B.quantize_fns(ctx, wl.shape, meta_fp16)
        self.reqs = synth.materialize(wl, dev, qk, qv, B.assemble_fn(ctx))
        for r in self.reqs:
            for ck in r.chunks:
                ck.meta_fp16 = int(ck.k_meta is not None and ck.k_meta.dtype == torch.float16)
        self._pack_payload(dev)
        sp = wl.select
        for r in self.reqs:
            r.kv_buf.zero_()
        self.tbl = B.RequestTable(self.reqs)
        Ts = [r.plan.T for r in self.reqs]
        self.ks = [sp.k_override if sp.k_override >= 0 else B.kvb_select_count(T, sp.ratio) for T in Ts]
        self.sel = B.SelectionTable(Ts, self.ks, [r.sel_capacity for r in self.reqs], dev)
        self.out = [torch.zeros_like(r.q) for r in self.reqs]
        self.q = [r.q for r in self.reqs]

    def _pack_payload(self, dev):
        """Moves every cached chunk's codes and metadata into one contiguous device arena (one H2D copy
        per step in the end-to-end measurement)."""
        tensors = []
        for r in self.reqs:
            for ck in r.chunks:
                for name in ("k_codes", "v_codes", "k_meta", "v_meta"):
                    t = getattr(ck, name)
                    if t is not None:
                        tensors.append((ck, name, t))
        total = sum((t.numel() * t.element_size() + 255) // 256 * 256 for _, _, t in tensors)
        self.arena = torch.empty(max(total, 256), dtype=torch.uint8, device=dev)
        off = 0
        for ck, name, t in tensors:
            nb = t.numel() * t.element_size()
            view = self.arena[off : off + nb].view(t.dtype).view(t.shape)
            view.copy_(t)
            setattr(ck, name, view)
            off += (nb + 255) // 256 * 256

    def device_bytes(self):
        n = self.arena.numel()
        for r, o in zip(self.reqs, self.out):
            n += 2 * r.kv_buf.numel() * 2 + 2 * r.q.numel() * 2
        return n


ONE_PASS = True  # stitch and deviation sums in one kernel (kvb_assemble_select); --path two-call uses the separate calls


def step(B, ctx, rep, sp, scale, events=None):
    if events:
        events[0].record()
    if ONE_PASS:
        B.kvb_assemble_select(ctx, rep.tbl, sp.ratio, sp.k_override, sp.seam_before, sp.seam_after, sp.which, rep.sel)
        if events:
            events[1].record()
    else:
        B.kvb_assemble(ctx, rep.tbl)
        if events:
            events[1].record()
        B.kvb_deviation_topk(ctx, rep.tbl, sp.ratio, sp.k_override, sp.seam_before, sp.seam_after, sp.which, rep.sel)
    if events:
        events[2].record()
    B.kvb_selective_attn(ctx, rep.tbl, rep.sel, rep.q, rep.out, scale)
    if events:
        events[3].record()


# --------------------------------------------------------------------------------------- oracle legs
def oracle_sample_seconds(wl, reqs_host, n_layers: int):
    """Runs the CPU oracle over the first n_layers layers of every request (all stages, all selected
    rows) and returns (seconds, threads).  Linear extrapolation in layers gives the full-path time."""
    import oracle

    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import helpers

    sh = wl.shape
    sub = synth.Shape(L=n_layers, Hq=sh.Hq, Hkv=sh.Hkv, d=sh.d, C=sh.C, theta=sh.theta, kv_dtype=sh.kv_dtype, int4_group=sh.int4_group)
    dtc = helpers.dt_code(sh)
    sp = wl.select
    t0 = time.perf_counter()
    for r in reqs_host:
        chunks = [synth.Chunk(c.plan, *(None if t is None else t[:n_layers] for t in (c.k_codes, c.v_codes, c.k_meta, c.v_meta))) for c in r.chunks]
        fresh = helpers.bits_of(r.fresh[:n_layers])
        kv = helpers.oracle_assemble_np(sub, r.plan, chunks, fresh)
        _, d32 = oracle.deviation(kv, fresh, dtc, sp.which)
        k = sp.k_override if sp.k_override >= 0 else oracle.select_count(r.plan.T, sp.ratio)
        rank = oracle.topk(d32, k)
        sel = oracle.seam_select(rank, [c.plan.new_pos for c in r.chunks], [c.plan.mode for c in r.chunks], r.plan.T, sp.seam_before, sp.seam_after)
        q = np.zeros((n_layers, len(sel), sh.Hq, sh.d), np.uint16)
        q[:] = helpers.bits_of(r.q[:n_layers, : len(sel)])
        oracle.attention(q, kv, sel, sh.Hq, dtc, 1.0 / math.sqrt(sh.d))
    return time.perf_counter() - t0, oracle.max_threads()


def host_copy(reqs):
    out = []
    for r in reqs:
        chunks = [synth.Chunk(c.plan, *(None if t is None else t.cpu() for t in (c.k_codes, c.v_codes, c.k_meta, c.v_meta))) for c in r.chunks]
        out.append(synth.Request(r.plan, chunks, r.fresh.cpu(), r.kv_buf.cpu(), r.q.cpu(), r.sel_capacity))
    return out


def reference_inputs(wl):
    """Inputs for the reference arm without a GPU: the oracle-side recipe on the host."""
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import helpers

    small = synth.Workload(wl.name, wl.seed, synth.Shape(L=1, Hq=wl.shape.Hq, Hkv=wl.shape.Hkv, kv_dtype=wl.shape.kv_dtype), wl.requests, wl.select)
    return small, helpers.materialize_with_oracle(small, "cpu")


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    small, reqs = reference_inputs(wl)
    tokens = sum(r.plan.T for r in reqs)
    L = wl.shape.L
    for _ in range(args.warmup):
        oracle_sample_seconds(small, reqs, 1)
    t = 0.0
    threads = 1
    for _ in range(args.steps):
        dt, threads = oracle_sample_seconds(small, reqs, 1)
        t += dt
    per_step_full = t / args.steps * L  # one of L layers was run per step
    value = tokens / per_step_full
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": per_step_full * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "tokens_per_step": tokens, "note": "CPU oracle; each step runs 1 of %d layers (all stages, all selected rows), time scaled by %d" % (L, L)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": "1 of %d layers per step, all stages" % L},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------------------- multi-rank glue
def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of device-measured times over all ranks (the slowest rank sets
    the job's time).  The path itself never communicates: ranks are independent replicas."""
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def job_throughput(world: int, tokens_per_rank_step: int, ms_per_step: float) -> float:
    """Whole-job tokens/s: every rank processes its own batch per step (weak scaling)."""
    return world * tokens_per_rank_step / (ms_per_step * 1e-3)


# --------------------------------------------------------------------------------------- main arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="kvb", choices=["kvb", "reference"])
    ap.add_argument("--workload", default="cfg1", choices=sorted(WORKLOADS))
    ap.add_argument("--replicas", type=int, default=0, help="independent copies rotated through (0 = auto)")
    ap.add_argument("--batch", type=int, default=1, help="requests per step: the workload's request list repeated this many times")
    ap.add_argument("--requests", type=int, default=0, help="cfg4 only: the ragged batch's first N requests instead of all 32")
    ap.add_argument("--path", default="one-pass", choices=["one-pass", "two-call"], help="kvb_assemble_select, or kvb_assemble + kvb_deviation_topk")
    ap.add_argument("--meta-fp16", action="store_true", help="cached chunks carry compact (binary16) scale/min pairs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    global ONE_PASS
    ONE_PASS = args.path == "one-pass"
    if args.requests > 0 and args.workload != "cfg4":
        ap.error("--requests applies to --workload cfg4")
    wl = synth.workload(WORKLOADS[args.workload], args.requests if args.requests > 0 else None)
    if args.requests > 0:  # a reduced ragged batch (profiling under a memory limit); not the workload the benchmark spec names
        wl = synth.Workload("%s_first%d" % (wl.name, args.requests), wl.seed, wl.shape, wl.requests, wl.select, wl.sigma_bulk, wl.sigma_seam, wl.seam_tokens)
    if args.batch > 1:
        wl = synth.Workload("%s_x%d" % (wl.name, args.batch), wl.seed, wl.shape, wl.requests * args.batch, wl.select, wl.sigma_bulk, wl.sigma_seam, wl.seam_tokens)
    if args.impl == "reference":
        run_reference(args, wl)
        return

    from paper_2608_21362_b200 import binding as B
    from paper_2608_21362_b200.build import build_library

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = "cuda:%d" % local
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device(dev))
    if rank == 0:
        build_library()
    if dist:
        dist.barrier()

    sh = wl.shape
    sp = wl.select
    scale = 1.0 / math.sqrt(sh.d)
    n_chunks = sum(len(r.chunks) for r in wl.requests)
    n_tok = sum(r.T for r in wl.requests)
    ctx = B.create_for_shape(sh, local, max_requests=len(wl.requests), max_chunks_total=n_chunks, max_tokens_total=n_tok)

    n_rep = args.replicas or {"cfg1": 8, "cfg2": 3, "cfg4": 1}[args.workload]
    reps = [Replica(B, ctx, wl, dev, 100 * rank + i, args.meta_fp16) for i in range(n_rep)]
    torch.cuda.synchronize()
    footprint = sum(r.device_bytes() for r in reps)

    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()

    def sync_all():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    for i in range(args.warmup):
        step(B, ctx, reps[i % n_rep], sp, scale)
    B.kvb_last_status(ctx)
    sync_all()

    # ---- the timed region: exactly K steps between two events.  Per-stage events are recorded in one
    #      step out of `stride` only: an event after every call sits between the calls' kernels (it breaks
    #      the dependent-launch chain and adds gaps: about 6 % on the short cfg1 step), so recording them
    #      everywhere would measure the instrumentation; the sampled steps are part of the timed region.
    stride = 8 if args.steps >= 40 else 1
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range((args.steps + stride - 1) // stride)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = B.kvb_launch_count(ctx)
    sampler.active = True
    t_wall0 = time.perf_counter()
    t_begin.record()
    for i in range(args.steps):
        step(B, ctx, reps[i % n_rep], sp, scale, ev[i // stride] if i % stride == 0 else None)
    t_end.record()
    sync_all()
    t_wall = time.perf_counter() - t_wall0
    sampler.active = False
    launches = B.kvb_launch_count(ctx) - launches0
    B.kvb_last_status(ctx)
    ms_total = t_begin.elapsed_time(t_end)  # device time from the first launch to the end of the last step
    n_stage = len(ev)
    stage_ms = [sum(e[j].elapsed_time(e[j + 1]) for e in ev) / n_stage for j in range(3)]

    # ---- end to end: every step's inputs start in pinned host memory and its results end there.
    #      With two or more replicas the copies are pipelined against the compute (H2D of step i+1 and
    #      D2H of step i-1 on their own streams, two device-side input/output sets); every step still
    #      moves all of its bytes inside the timed region.
    e2e = None
    if not args.no_e2e:
        slots = reps[:2] if len(reps) >= 2 else reps[:1]
        s_in, s_out, s_cmp = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
        io = []
        for rep in slots:
            devs_in = [rep.arena] + [r.fresh for r in rep.reqs] + rep.q
            pins_in = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t) for t in devs_in]
            devs_out = rep.out + rep.sel.sel + [rep.sel.n_sel]
            pins_out = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in devs_out]
            ev = {k: torch.cuda.Event() for k in ("in", "cmp", "out")}
            for e in ev.values():
                e.record(s_cmp)
            io.append((rep, devs_in, pins_in, devs_out, pins_out, ev))
        h2d = sum(t.numel() * t.element_size() for t in io[0][1])
        d2h = sum(t.numel() * t.element_size() for t in io[0][3])

        def e2e_step(i):
            rep, devs_in, pins_in, devs_out, pins_out, ev = io[i % len(io)]
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev["cmp"])  # the previous step on this slot has consumed its inputs
                for p, d in zip(pins_in, devs_in):
                    d.copy_(p, non_blocking=True)
                ev["in"].record(s_in)
            s_cmp.wait_event(ev["in"])
            s_cmp.wait_event(ev["out"])  # the previous results of this slot have left the device
            step(B, ctx, rep, sp, scale)
            ev["cmp"].record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev["cmp"])
                for p, d in zip(pins_out, devs_out):
                    p.copy_(d, non_blocking=True)
                ev["out"].record(s_out)

        def drain():
            for _, _, _, _, _, ev in io:
                s_cmp.wait_event(ev["out"])
                s_cmp.wait_event(ev["in"])

        n_e2e = max(4, min(args.steps, 20))
        for i in range(4):
            e2e_step(i)
        drain()
        sync_all()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(n_e2e):
            e2e_step(i)
        drain()
        b.record()
        sync_all()
        e2e_ms = a.elapsed_time(b) / n_e2e
        e2e = {"ms_per_step": e2e_ms, "h2d": h2d, "d2h": d2h, "steps": n_e2e, "pipelined": len(io) > 1}
    sampler.stop()

    # ---- algorithmic work per step
    pair_bytes = 4 if args.meta_fp16 else 8
    asm_bytes = sum(synth.assemble_bytes(sh, r.plan, pair_bytes) for r in reps[0].reqs)
    dev_bytes = sum(synth.deviation_bytes(sh, r.plan, sp.which) for r in reps[0].reqs)
    flops = []
    for rep in reps:
        f = 0
        ns = rep.sel.n_sel.cpu().numpy()
        for i, r in enumerate(rep.reqs):
            f += synth.attention_flops(sh, rep.sel.sel[i].cpu().numpy()[: ns[i]])
        flops.append(f)
    attn_flops = float(np.mean(flops))

    if dist:
        t = max_over_ranks([ms_total] + stage_ms + ([e2e["ms_per_step"]] if e2e else [0.0]), dist, dev)
        ms_total, stage_ms = t[0], t[1:4]
        if e2e:
            e2e["ms_per_step"] = t[4]

    peaks = load_peaks()
    ms_step = ms_total / args.steps
    value = job_throughput(world, n_tok, ms_step)
    long_run = ms_total > 1000.0
    tensor_peak = peaks["bf16_sustained"] if long_run else peaks["bf16_burst"]
    attn_stage = {"bound": "tensor", "ms": stage_ms[2], "achieved": attn_flops / stage_ms[2] / 1e9, "peak": tensor_peak, "unit": "TFLOP/s", "algorithmic_flops": attn_flops}
    if ONE_PASS:  # stitch + deviation sums + selection behind one call
        one_bytes = sum(synth.one_pass_bytes(sh, r.plan, sp.which, pair_bytes) for r in reps[0].reqs)
        ms01 = stage_ms[0] + stage_ms[1]
        stages = {
            "assemble_select": {"bound": "hbm", "ms": ms01, "achieved": one_bytes / ms01 / 1e6, "peak": peaks["hbm_gbs"], "unit": "GB/s", "algorithmic_bytes": one_bytes,
                                "two_call_bytes": asm_bytes + dev_bytes},
            "selective_attn": attn_stage,
        }
    else:
        stages = {
            "assemble": {"bound": "hbm", "ms": stage_ms[0], "achieved": asm_bytes / stage_ms[0] / 1e6, "peak": peaks["hbm_gbs"], "unit": "GB/s", "algorithmic_bytes": asm_bytes},
            "deviation_topk": {"bound": "hbm", "ms": stage_ms[1], "achieved": dev_bytes / stage_ms[1] / 1e6, "peak": peaks["hbm_gbs"], "unit": "GB/s", "algorithmic_bytes": dev_bytes},
            "selective_attn": attn_stage,
        }
    for s in stages.values():
        s["frac"] = s["achieved"] / s["peak"]
        # context only: fraction of the nominal figure (8 TB/s HBM3e, 2250 TFLOP/s dense bf16)
        s["frac_of_nominal"] = s["achieved"] / (8000.0 if s["bound"] == "hbm" else 2250.0)
    top = max(stages, key=lambda k: stages[k]["ms"])
    roof = {k: stages[top][k] for k in ("bound", "achieved", "peak", "unit", "frac")}
    # dram__bytes_read.sum + dram__bytes_write.sum of one launch, from the committed ncu captures
    # (profiles/cfg1_launches_and_kernels.md, profiles/cfg2_kernels.md); null where none was taken
    ncu_traffic = {
        ("cfg1_qwen3b_2k_int8", "selective_attn"): 211.9e6, ("cfg1_qwen3b_2k_int8", "assemble"): 67.6e6,
        ("cfg1_qwen3b_2k_int8", "assemble_select"): 125.6e6,
        ("cfg1_qwen3b_2k_int8", "deviation_topk"): 154.2e6, ("cfg2_long_int4_8k", "selective_attn"): 730.0e6,
        ("cfg2_long_int4_8k", "assemble_select"): 646.8e6,
        ("cfg2_long_int4_8k", "assemble"): 381.0e6, ("cfg2_long_int4_8k", "deviation_topk"): 608.2e6,
    }
    roof.update({"kernel": top, "traffic": ncu_traffic.get((wl.name, top)), "peak_source": "%s (%s)" % (peaks["source"], "sustained" if (top == "selective_attn" and long_run) else "burst/copy"),
                 "timing": "CUDA events around the C-ABI call of the stage in %d of the timed steps (one in %d); ms_per_step and value come from two events around all K steps" % (n_stage, stride)})

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if sh.kv_dtype == "bf16" else "fp16", "data": "synthetic",
        "config": {
            "workload": wl.name, "path": "kvb_assemble_select + kvb_selective_attn" if ONE_PASS else "kvb_assemble + kvb_deviation_topk + kvb_selective_attn",
            "metadata": "binary16 (scale, min) pairs" if args.meta_fp16 else "float32 (scale, min) pairs",
            "requests_per_step": len(wl.requests), "tokens_per_step": n_tok, "layers": sh.L, "q_heads": sh.Hq,
            "kv_heads": sh.Hkv, "head_dim": sh.d, "chunk_tokens": sh.C, "select_ratio": sp.ratio, "seam_window": [sp.seam_before, sp.seam_after],
            "parallelism": "replicas only (one independent stream of requests per GPU)" if world > 1 else "single GPU",
            "l2": "inputs larger than L2: %d replicas rotated, %.0f MB resident" % (n_rep, footprint / 1e6),
        },
        "roofline": roof, "stages": stages, "gpu_launches": int(launches),
        "clocks": sampler.summary(), "wall_s_timed": t_wall,
    }
    if e2e:
        line["e2e"] = {"value": job_throughput(world, n_tok, e2e["ms_per_step"]), "unit": UNIT, "h2d_bytes_per_step": e2e["h2d"],
                       "d2h_bytes_per_step": e2e["d2h"], "ms_per_step": e2e["ms_per_step"], "steps": e2e["steps"],
                       "copies": "pipelined on separate streams over 2 device-side sets" if e2e["pipelined"] else "in line with the compute"}

    # ---- CPU oracle beside it (rank 0, N=1 only): bounded sample of the same workload
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        order = sorted(range(len(reps[0].reqs)), key=lambda i: reps[0].reqs[i].plan.T)
        if n_tok > 20000:  # a batch: the four shortest requests only
            order = order[:4]
        reqs_host = host_copy([reps[0].reqs[i] for i in order])
        # one layer first to calibrate, then as many layers as make about 12 s of CPU work
        t1, threads = oracle_sample_seconds(wl, reqs_host, 1)
        n_l = max(1, min(sh.L, int(round(12.0 / max(t1, 1e-3)))))
        secs = t1 if n_l == 1 else oracle_sample_seconds(wl, reqs_host, n_l)[0]
        tok_s = sum(r.plan.T for r in reqs_host)
        line["cpu_baseline"] = {
            "value": tok_s / (secs * sh.L / n_l), "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": "%d request(s), %d tokens, %d of %d layers, all stages and all selected rows; %.1f s measured, scaled by layers" % (len(reqs_host), tok_s, n_l, sh.L, secs),
        }
        if t1 * threads <= 12.0:  # one core as well, where a single layer stays within a few seconds
            import oracle

            oracle.set_threads(1)
            s1 = oracle_sample_seconds(wl, reqs_host, 1)[0]
            oracle.set_threads(threads)
            line["cpu_baseline"]["value_1_core"] = tok_s / (s1 * sh.L)
    B.kvb_destroy(ctx)
    if rank == 0:
        print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
