#!/usr/bin/env python
"""Benchmark of the KV-chunk stitching path on B200.

A step is one pass of the whole path over one batch of synthetic requests:
    kvb_assemble_select (stitch + deviation sums in one kernel, then the selection) -> kvb_selective_attn
(`--path two-call`: kvb_assemble -> kvb_deviation_topk -> kvb_selective_attn, the same work in three calls).

  python bench.py --gpus N --steps K --warmup W [--workload all|cfg1|cfg2|cfg3|cfg4] [--impl reference]
                  [--stage path|patch|importance|quantize]

The headline workload is the largest configuration, the 32-request ragged batch (cfg4).  With the
default `--workload all` (one GPU) the same line carries, under `per_config`, the 2048-token int8
prompt (cfg1), the 8192-token int4 prompt (cfg2) and the stand-alone selective attention of its 1229
selected rows (cfg3).  `--stage` times one of the kernels next to the path instead (patch,
importance score, quantiser) and prints its own line.

Timing: `value` / `ms_per_step` come from two CUDA events around exactly K steps with nothing
recorded in between; a short region is repeated until half a second of device time has passed and the
median region is reported.  The per-stage times come from a separate instrumented pass afterwards.

Prints one JSON line (rank 0).  `--impl reference` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import hashlib
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
WORKLOADS = {"cfg1": 1, "cfg2": 2, "cfg3": 3, "cfg4": 4}
HEADLINE = "cfg4"
REPLICAS = {"cfg1": 8, "cfg2": 3, "cfg3": 3, "cfg4": 1}  # independent copies rotated so that a step's inputs never sit in L2
MIN_REGION_MS = 500.0  # a K-step region shorter than this is repeated until this much device time has passed
CSRC = os.path.join(ROOT, "paper_2608_21362_b200", "csrc")


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

    def begin(self):
        """Starts a new record (one per measured workload)."""
        self.samples, self.reasons = [], set()
        self.active = True

    def end(self):
        self.active = False
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
        bq = B.BatchedQuantizer(ctx, wl.shape, meta_fp16)  # the chunks of a request are quantised by one call
        self.reqs = synth.materialize(wl, dev, bq.quantize_k, bq.quantize_v, bq.assemble)
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


def step_attention_only(B, ctx, rep, sp, scale, events=None):
    """cfg3: the selective attention alone, on a buffer and a selection prepared beforehand."""
    if events:
        for e in events[:3]:
            e.record()
    B.kvb_selective_attn(ctx, rep.tbl, rep.sel, rep.q, rep.out, scale)
    if events:
        events[3].record()


# --------------------------------------------------------------------------------------- oracle legs
def oracle_sample_seconds(wl, reqs_host, n_layers: int):
    """Runs the CPU oracle over the first n_layers layers of every request (all stages, all selected
    rows) and returns (seconds, threads).  Linear extrapolation in layers gives the full-path time."""
    import oracle
    import oracle_glue as glue

    sh = wl.shape
    sub = synth.Shape(L=n_layers, Hq=sh.Hq, Hkv=sh.Hkv, d=sh.d, C=sh.C, theta=sh.theta, kv_dtype=sh.kv_dtype, int4_group=sh.int4_group)
    dtc = glue.dt_code(sh)
    sp = wl.select
    t0 = time.perf_counter()
    for r in reqs_host:
        chunks = [synth.Chunk(c.plan, *(None if t is None else t[:n_layers] for t in (c.k_codes, c.v_codes, c.k_meta, c.v_meta))) for c in r.chunks]
        fresh = glue.bits_of(r.fresh[:n_layers])
        kv = glue.oracle_assemble_np(sub, r.plan, chunks, fresh)
        _, d32 = oracle.deviation(kv, fresh, dtc, sp.which)
        k = sp.k_override if sp.k_override >= 0 else oracle.select_count(r.plan.T, sp.ratio)
        rank = oracle.topk(d32, k)
        sel = oracle.seam_select(rank, [c.plan.new_pos for c in r.chunks], [c.plan.mode for c in r.chunks], r.plan.T, sp.seam_before, sp.seam_after)
        q = np.zeros((n_layers, len(sel), sh.Hq, sh.d), np.uint16)
        q[:] = glue.bits_of(r.q[:n_layers, : len(sel)])
        oracle.attention(q, kv, sel, sh.Hq, dtc, 1.0 / math.sqrt(sh.d))
    return time.perf_counter() - t0, oracle.max_threads()


def host_copy(reqs):
    out = []
    for r in reqs:
        chunks = [synth.Chunk(c.plan, *(None if t is None else t.cpu() for t in (c.k_codes, c.v_codes, c.k_meta, c.v_meta))) for c in r.chunks]
        out.append(synth.Request(r.plan, chunks, r.fresh.cpu(), r.kv_buf.cpu(), r.q.cpu(), r.sel_capacity))
    return out


def oracle_sample_ids(wl):
    """The bounded sample of a workload the CPU legs run: every request of a single-prompt workload,
    the four shortest requests of a batch."""
    order = sorted(range(len(wl.requests)), key=lambda i: wl.requests[i].T)
    return order[:4] if sum(r.T for r in wl.requests) > 20000 else order


def config_dict(wl, path, meta_fp16, world, n_replicas, attention_pairs=False):
    """The `config` object of the JSON line; both arms (kvb and reference) print the same one."""
    sh, sp = wl.shape, wl.select
    cfg = {
        "workload": wl.name, "path": path,
        "metadata": "binary16 (scale, min) pairs" if meta_fp16 else "float32 (scale, min) pairs",
        "requests_per_step": len(wl.requests), "tokens_per_step": sum(r.T for r in wl.requests), "layers": sh.L, "q_heads": sh.Hq,
        "kv_heads": sh.Hkv, "head_dim": sh.d, "chunk_tokens": sh.C, "select_ratio": sp.ratio, "seam_window": [sp.seam_before, sp.seam_after],
        "parallelism": "replicas only (one independent stream of requests per GPU)" if world > 1 else "single GPU",
    }
    if attention_pairs:
        cfg["attention"] = "paired-CTA form (debug option attention_cta_pairs)"
    cfg["l2"] = "inputs larger than L2, no flush: %s" % ("the batch itself exceeds it" if n_replicas == 1 else "%d independent replicas of the batch rotated" % n_replicas)
    return cfg


PATH_NAMES = {True: "kvb_assemble_select + kvb_selective_attn", False: "kvb_assemble + kvb_deviation_topk + kvb_selective_attn"}


def run_reference(args, key, wl):
    """The reference arm: the CPU oracle, as it stands, on a bounded sample of the headline workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle_glue as glue

    ids = oracle_sample_ids(wl)
    small = synth.Workload(wl.name, wl.seed, synth.Shape(L=1, Hq=wl.shape.Hq, Hkv=wl.shape.Hkv, kv_dtype=wl.shape.kv_dtype), wl.requests, wl.select)
    reqs = glue.materialize_with_oracle(small, "cpu", ids)
    tokens = sum(r.plan.T for r in reqs)
    L = wl.shape.L
    for _ in range(args.warmup):
        oracle_sample_seconds(small, reqs, 1)
    t = 0.0
    threads = 1
    for _ in range(args.steps):
        dt, threads = oracle_sample_seconds(small, reqs, 1)
        t += dt
    # A token of the metric is all L layers of one position; a step runs one layer of the sample's
    # positions, i.e. tokens / L token-equivalents, and ms_per_step is the time it really took.
    per_step = t / args.steps
    value = (tokens / L) / per_step
    sample = "%d request(s), %d tokens, 1 of %d layers per step (all stages, all selected rows) = %.1f token-equivalents per step" % (len(reqs), tokens, L, tokens / L)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(wl, PATH_NAMES[ONE_PASS], args.meta_fp16, 1, args.replicas or REPLICAS.get(key, 1)),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
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


# --------------------------------------------------------------------------------------- ncu traffic records
def recorded_traffic(workload: str, stage: str, units_now: float):
    """dram read+write bytes of one launch of the stage's dominant kernel, from the committed ncu
    records, or None.  A record names the kernel's source file and its SHA-256 at capture time: when
    the file has changed since, the record no longer describes the kernel and None is returned.  A
    record taken on a reduced case carries the units (tokens) it processed and is scaled."""
    p = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    if not os.path.exists(p):
        return None, None
    for rec in json.load(open(p))["records"]:
        if rec["workload"] != workload or rec["stage"] != stage:
            continue
        src = os.path.join(CSRC, rec["source"])
        if not os.path.exists(src) or hashlib.sha256(open(src, "rb").read()).hexdigest() != rec["source_sha256"]:
            return None, "record of commit %s predates the current %s" % (rec.get("commit", "?"), rec["source"])
        scale = units_now / rec["units"] if rec.get("units") else 1.0
        note = "ncu capture at commit %s on %s" % (rec.get("commit", "?"), rec.get("captured_on", workload))
        if abs(scale - 1.0) > 1e-9:
            note += ", scaled by %.3f (units processed)" % scale
        return rec["dram_bytes_per_launch"] * scale, note
    return None, None


# --------------------------------------------------------------------------------------- one workload
class Runner:
    def __init__(self, args, B, dist, rank, world, local, sampler):
        self.args, self.B, self.dist, self.rank, self.world, self.local, self.sampler = args, B, dist, rank, world, local, sampler
        self.dev = "cuda:%d" % local
        self.peaks = load_peaks()

    def sync_all(self):
        torch.cuda.synchronize()
        if self.dist:
            self.dist.barrier()
            torch.cuda.synchronize()

    def build(self, key, wl):
        B, args = self.B, self.args
        n_chunks = sum(len(r.chunks) for r in wl.requests)
        n_tok = sum(r.T for r in wl.requests)
        ctx = B.create_for_shape(wl.shape, self.local, max_requests=len(wl.requests), max_chunks_total=n_chunks, max_tokens_total=n_tok)
        if args.attention_pairs:
            B.kvb_set_debug_option(ctx, "attention_cta_pairs", 1)
        if args.attention_two_tiles:
            B.kvb_set_debug_option(ctx, "attention_two_tiles", 1)
        n_rep = args.replicas or REPLICAS[key]
        reps = [Replica(B, ctx, wl, self.dev, 100 * self.rank + i, args.meta_fp16) for i in range(n_rep)]
        if key == "cfg3":  # the buffer and the selection the attention runs on, prepared outside the timed region
            sp = wl.select
            for rep in reps:
                B.kvb_assemble_select(ctx, rep.tbl, sp.ratio, sp.k_override, sp.seam_before, sp.seam_after, sp.which, rep.sel)
            B.kvb_last_status(ctx)
        torch.cuda.synchronize()
        return ctx, reps

    def measure(self, key, wl, headline):
        """Times one workload.  Returns the result dict (times are the max over ranks)."""
        B, args, dist = self.B, self.args, self.dist
        sh, sp = wl.shape, wl.select
        scale = 1.0 / math.sqrt(sh.d)
        n_tok = sum(r.T for r in wl.requests)
        ctx, reps = self.build(key, wl)
        n_rep = len(reps)
        footprint = sum(r.device_bytes() for r in reps)
        do_step = step_attention_only if key == "cfg3" else step
        K = args.steps

        for i in range(args.warmup):
            do_step(B, ctx, reps[i % n_rep], sp, scale)
        B.kvb_last_status(ctx)
        self.sync_all()

        # ---- the timed regions: exactly K steps between two events, nothing recorded in between.  A
        #      region shorter than MIN_REGION_MS is repeated (same K) until that much device time has
        #      passed; the median region is reported, so that the clock sampler sees the whole of it.
        self.sampler.begin()
        regions, launches, t_wall0, it = [], 0, time.perf_counter(), 0
        while True:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            l0 = B.kvb_launch_count(ctx)
            a.record()
            for _ in range(K):
                do_step(B, ctx, reps[it % n_rep], sp, scale)
                it += 1
            b.record()
            self.sync_all()
            launches = B.kvb_launch_count(ctx) - l0
            ms = a.elapsed_time(b)
            if dist:
                ms = max_over_ranks([ms], dist, self.dev)[0]
            regions.append(ms)
            if sum(regions) >= args.min_region_ms or len(regions) >= 400:
                break
        t_wall = time.perf_counter() - t_wall0
        clocks = self.sampler.end()
        B.kvb_last_status(ctx)
        ms_region = float(np.median(regions))
        ms_step = ms_region / K

        # ---- the instrumented pass (not part of `value`): an event after every call gives the stage times.
        #      The events sit between the calls' kernels (they break the dependent-launch chain), so these
        #      steps are a little slower than the clean ones: their sum is reported next to ms_per_step.
        n_inst = max(3, min(K, 16))
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(n_inst)]
        for i in range(n_inst):
            do_step(B, ctx, reps[(it + i) % n_rep], sp, scale, ev[i])
        self.sync_all()
        B.kvb_last_status(ctx)
        stage_ms = [sum(e[j].elapsed_time(e[j + 1]) for e in ev) / n_inst for j in range(3)]
        if dist:
            stage_ms = max_over_ranks(stage_ms, dist, self.dev)

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

        peaks = self.peaks
        long_run = ms_region > 1000.0
        tensor_peak = peaks["bf16_sustained"] if long_run else peaks["bf16_burst"]
        stages = {}
        if key != "cfg3":
            if ONE_PASS:  # stitch + deviation sums + selection behind one call
                one_bytes = sum(synth.one_pass_bytes(sh, r.plan, sp.which, pair_bytes) for r in reps[0].reqs)
                ms01 = stage_ms[0] + stage_ms[1]
                stages["assemble_select"] = {"bound": "hbm", "ms": ms01, "achieved": one_bytes / ms01 / 1e6, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                             "algorithmic_bytes": one_bytes, "two_call_bytes": asm_bytes + dev_bytes}
            else:
                stages["assemble"] = {"bound": "hbm", "ms": stage_ms[0], "achieved": asm_bytes / stage_ms[0] / 1e6, "peak": peaks["hbm_gbs"], "unit": "GB/s", "algorithmic_bytes": asm_bytes}
                stages["deviation_topk"] = {"bound": "hbm", "ms": stage_ms[1], "achieved": dev_bytes / stage_ms[1] / 1e6, "peak": peaks["hbm_gbs"], "unit": "GB/s", "algorithmic_bytes": dev_bytes}
        stages["selective_attn"] = {"bound": "tensor", "ms": stage_ms[2], "achieved": attn_flops / stage_ms[2] / 1e9, "peak": tensor_peak, "unit": "TFLOP/s",
                                    "algorithmic_flops": attn_flops, "peak_kind": "sustained" if long_run else "burst"}
        for s in stages.values():
            s["frac"] = s["achieved"] / s["peak"]
            # context only: fraction of the nominal figure (8 TB/s HBM3e, 2250 TFLOP/s dense bf16)
            s["frac_of_nominal"] = s["achieved"] / (8000.0 if s["bound"] == "hbm" else 2250.0)
        top = max(stages, key=lambda k: stages[k]["ms"])
        roof = {k: stages[top][k] for k in ("bound", "achieved", "peak", "unit", "frac")}
        traffic, traffic_note = recorded_traffic(wl.name, top, n_tok)
        roof.update({"kernel": top, "traffic": traffic, "traffic_source": traffic_note,
                     "peak_source": "%s (%s)" % (peaks["source"], stages[top].get("peak_kind", "copy")),
                     "timing": "CUDA events around the stage's C-ABI call in a separate instrumented pass of %d steps after the timed region" % n_inst})
        res = {
            "workload": wl.name, "ms_per_step": ms_step, "value": job_throughput(self.world, n_tok, ms_step), "tokens_per_step": n_tok,
            "regions": {"count": len(regions), "steps_each": K, "ms_median": ms_region, "ms_min": float(min(regions)), "ms_max": float(max(regions))},
            "instrumented_ms_per_step": sum(stage_ms), "stages": stages, "roofline": roof, "gpu_launches": int(launches), "clocks": clocks,
            "wall_s_timed": t_wall, "l2": "inputs larger than L2: %d replica(s) rotated, %.0f MB resident" % (n_rep, footprint / 1e6),
        }
        if headline:
            if not args.no_e2e:
                e2e_reps = reps
                if len(reps) == 1 and key != "cfg3":
                    # a second device-side set, so that the copies of one step run under the compute and the
                    # copies of its neighbours (where the GPU and the host have the room for it)
                    free_dev, _ = torch.cuda.mem_get_info(self.dev)
                    if free_dev > 1.25 * footprint:
                        e2e_reps = reps + [Replica(B, ctx, wl, self.dev, 100 * self.rank + 1, args.meta_fp16)]
                res["e2e"] = self.end_to_end(ctx, e2e_reps, do_step, sp, scale, n_tok)
                del e2e_reps
            if self.rank == 0 and self.world == 1 and not args.no_cpu_baseline and key != "cfg3":
                res["cpu_baseline"] = self.cpu_baseline(wl, reps[0])
        B.kvb_destroy(ctx)
        del reps
        torch.cuda.empty_cache()
        return res

    # ---- end to end: every step's inputs start in pinned host memory and its results end there.
    #      With two or more replicas the copies are pipelined against the compute (H2D of step i+1 and
    #      D2H of step i-1 on their own streams, two device-side input/output sets); every step still
    #      moves all of its bytes inside the timed region.
    def end_to_end(self, ctx, reps, do_step, sp, scale, n_tok):
        B, args = self.B, self.args
        slots = reps[:2] if len(reps) >= 2 else reps[:1]

        def io_tensors(rep):
            return [rep.arena] + [r.fresh for r in rep.reqs] + rep.q, rep.out + rep.sel.sel + [rep.sel.n_sel]

        bytes_of = lambda sl: sum(t.numel() * t.element_size() for rep in sl for ts in io_tensors(rep) for t in ts)
        try:
            import psutil

            avail = psutil.virtual_memory().available
        except Exception:
            avail = None
        local_world = int(os.environ.get("LOCAL_WORLD_SIZE", str(self.world)))
        if avail is not None and len(slots) > 1 and bytes_of(slots) * local_world > 0.5 * avail:
            slots = slots[:1]  # pinned buffers for one set only: the copies then run in line with the compute
        need = bytes_of(slots)
        if avail is not None and need * local_world > 0.5 * avail:
            return {"value": None, "unit": UNIT, "skipped": "pinned host buffers of %.1f GB x %d ranks exceed half of the host's free memory" % (need / 1e9, local_world)}
        s_in, s_out, s_cmp = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
        io = []
        for rep in slots:
            devs_in, devs_out = io_tensors(rep)
            pins_in = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t) for t in devs_in]
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
            do_step(B, ctx, rep, sp, scale)
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

        big = h2d + d2h > 4e9  # a step that moves tens of GB over PCIe takes about a second
        # pipelined steps: enough of them that filling and draining the two-deep pipeline weigh little
        n_warm, n_e2e = ((1, 3) if len(io) == 1 else (2, 8)) if big else (4, max(4, min(args.steps, 20)))
        for i in range(n_warm):
            e2e_step(i)
        drain()
        self.sync_all()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(n_e2e):
            e2e_step(i)
        drain()
        b.record()
        self.sync_all()
        ms = a.elapsed_time(b) / n_e2e
        if self.dist:
            ms = max_over_ranks([ms], self.dist, self.dev)[0]
        return {"value": job_throughput(self.world, n_tok, ms), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": ms, "steps": n_e2e,
                "copies": "pipelined on separate streams over 2 device-side sets" if len(io) > 1 else "in line with the compute"}

    # ---- CPU oracle beside it (rank 0, N=1 only): bounded sample of the same workload
    def cpu_baseline(self, wl, rep):
        sh = wl.shape
        ids = oracle_sample_ids(wl)
        reqs_host = host_copy([rep.reqs[i] for i in ids])
        # one layer first to calibrate, then as many layers as make about 12 s of CPU work
        t1, threads = oracle_sample_seconds(wl, reqs_host, 1)
        n_l = max(1, min(sh.L, int(round(12.0 / max(t1, 1e-3)))))
        secs = t1 if n_l == 1 else oracle_sample_seconds(wl, reqs_host, n_l)[0]
        tok_s = sum(r.plan.T for r in reqs_host)
        out = {
            "value": tok_s / (secs * sh.L / n_l), "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": "%d request(s), %d tokens, %d of %d layers, all stages and all selected rows; %.1f s measured, scaled by layers" % (len(reqs_host), tok_s, n_l, sh.L, secs),
        }
        if t1 * threads <= 12.0:  # one core as well, where a single layer stays within a few seconds
            import oracle

            oracle.set_threads(1)
            s1 = oracle_sample_seconds(wl, reqs_host, 1)[0]
            oracle.set_threads(threads)
            out["value_1_core"] = tok_s / (s1 * sh.L)
        return out

    # ---- the kernels next to the path: one HBM-bound kernel each, algorithmic GB/s against the copy peak
    def measure_stage(self, stage, key, wl):
        B, args = self.B, self.args
        sh, sp = wl.shape, wl.select
        ctx, reps = self.build(key, wl)
        n_rep = len(reps)
        B.kvb_destroy(ctx)  # a context sized for the stage's own calls (128 quantise jobs)
        n_chunks = max(128, sum(len(r.chunks) for r in wl.requests))
        ctx = B.create_for_shape(sh, self.local, max_requests=len(wl.requests), max_chunks_total=n_chunks, max_tokens_total=sum(r.T for r in wl.requests))
        for rep in reps:  # the selection and the stitched buffer the stage works on
            B.kvb_assemble_select(ctx, rep.tbl, sp.ratio, sp.k_override, sp.seam_before, sp.seam_after, sp.which, rep.sel)
        B.kvb_last_status(ctx)
        row_bytes = sh.Hkv * sh.d * 2
        if stage == "patch":
            n_sel = [int(x) for x in reps[0].sel.n_sel.cpu()]
            alg = sum(n_sel) * sh.L * 2 * row_bytes * 2  # fresh K and V rows read, buffer rows written
            call = lambda rep: B.kvb_patch(ctx, rep.tbl, rep.sel)
            passage = "Algorithm 2 step 4 (kvb_patch), %d selected rows" % sum(n_sel)
        elif stage == "importance":
            for rep in reps:
                rep.imp = [torch.zeros(len(r.chunks), dtype=torch.float32, device=self.dev) for r in rep.reqs]
            alg = sum(r.plan.T for r in reps[0].reqs) * sh.L * row_bytes  # every key row once
            call = lambda rep: B.kvb_chunk_importance(ctx, rep.tbl, rep.imp)
            passage = "Eq. 7 (kvb_chunk_importance)"
        elif stage == "quantize":
            # cache population of 128 chunks (a 16K-token prompt), keys and values, one call
            n_jobs = 128
            bits = args.quantize_bits
            gk, gv = (1, 1) if bits == 8 else (sh.C // sh.int4_group, sh.d // sh.int4_group)  # groups per channel / per row
            g = torch.Generator(device=self.dev).manual_seed(5)
            for rep in reps:
                rep.qjobs = []
                for _ in range(n_jobs):
                    kx = torch.randn((sh.L, sh.C, sh.Hkv, sh.d), generator=g, device=self.dev).to(sh.torch_dtype)
                    vx = torch.randn((sh.L, sh.C, sh.Hkv, sh.d), generator=g, device=self.dev).to(sh.torch_dtype)
                    mk = lambda *shape: torch.empty(shape, dtype=torch.uint8, device=self.dev)
                    rep.qjobs.append(dict(k=kx, v=vx, k_codes=mk(sh.L, sh.C, sh.Hkv, sh.d * bits // 8), v_codes=mk(sh.L, sh.C, sh.Hkv, sh.d * bits // 8),
                                          k_meta=torch.empty((sh.L, gk, sh.Hkv, sh.d, 2), device=self.dev),
                                          v_meta=torch.empty((sh.L, sh.C, sh.Hkv, gv, 2), device=self.dev), bits=bits,
                                          unrotate_from=(sh.C * len(rep.qjobs) if args.quantize_unrotate else -1)))
            E = sh.Hkv * sh.d
            alg = n_jobs * sh.L * (2 * sh.C * E * 2 + 2 * sh.C * E * bits // 8 + gk * E * 8 + sh.C * sh.Hkv * gv * 8)  # 16-bit rows read, codes and metadata written
            for rep in reps:
                rep.qtable = B.QuantizeTable(rep.qjobs)  # marshalled once, like the request tables
            call = lambda rep: B.kvb_quantize_chunks(ctx, rep.qtable)
            passage = "Eq. 6 forward (kvb_quantize_chunks), %d chunks x (keys + values), int%d%s" % (
                n_jobs, bits, ", keys rotated back to position 0 (Eq. 3)" if args.quantize_unrotate else "")
        else:
            raise SystemExit("unknown stage %s" % stage)
        for i in range(max(args.warmup, 3)):
            call(reps[i % n_rep])
        self.sync_all()
        self.sampler.begin()
        regions, it = [], 0
        while (not regions or sum(regions) < args.min_region_ms) and len(regions) < 400:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(args.steps):
                call(reps[it % n_rep])
                it += 1
            b.record()
            self.sync_all()
            regions.append(a.elapsed_time(b))
        clocks = self.sampler.end()
        B.kvb_last_status(ctx)
        ms = float(np.median(regions)) / args.steps
        gbs = alg / ms / 1e6
        B.kvb_destroy(ctx)
        return {"stage": stage, "computes": passage, "workload": wl.name, "ms_per_call": ms, "algorithmic_bytes": alg, "achieved": gbs, "unit": "GB/s",
                "peak": self.peaks["hbm_gbs"], "frac": gbs / self.peaks["hbm_gbs"], "frac_of_nominal": gbs / 8000.0, "clocks": clocks,
                "regions": len(regions), "l2": "%d replicas rotated" % n_rep}


def named_workload(key, args):
    wl = synth.workload(WORKLOADS[key], args.requests if (args.requests > 0 and key == "cfg4") else None)
    if args.requests > 0 and key == "cfg4":  # a reduced ragged batch (profiling under a memory limit); not the workload the benchmark spec names
        wl = synth.Workload("%s_first%d" % (wl.name, args.requests), wl.seed, wl.shape, wl.requests, wl.select, wl.sigma_bulk, wl.sigma_seam, wl.seam_tokens)
    if args.batch > 1:
        wl = synth.Workload("%s_x%d" % (wl.name, args.batch), wl.seed, wl.shape, wl.requests * args.batch, wl.select, wl.sigma_bulk, wl.sigma_seam, wl.seam_tokens)
    return wl


# --------------------------------------------------------------------------------------- main arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="kvb", choices=["kvb", "reference"])
    ap.add_argument("--workload", default="all", choices=["all"] + sorted(WORKLOADS),
                    help="all: the ragged batch (cfg4) as the headline plus cfg1, cfg2, cfg3 under per_config; or one workload alone")
    ap.add_argument("--stage", default="path", choices=["path", "patch", "importance", "quantize"], help="time one kernel next to the path instead of the path")
    ap.add_argument("--replicas", type=int, default=0, help="independent copies rotated through (0 = auto)")
    ap.add_argument("--batch", type=int, default=1, help="requests per step: the workload's request list repeated this many times")
    ap.add_argument("--requests", type=int, default=0, help="cfg4 only: the ragged batch's first N requests instead of all 32")
    ap.add_argument("--path", default="one-pass", choices=["one-pass", "two-call"], help="kvb_assemble_select, or kvb_assemble + kvb_deviation_topk")
    ap.add_argument("--meta-fp16", action="store_true", help="cached chunks carry compact (binary16) scale/min pairs")
    ap.add_argument("--min-region-ms", type=float, default=MIN_REGION_MS,
                    help="a K-step region shorter than this is repeated until this much device time has passed (0: one region, for profiler runs)")
    ap.add_argument("--attention-pairs", action="store_true",
                    help="run kvb_selective_attn in its paired-CTA form (the context's attention_cta_pairs option; measured slower, not the default)")
    ap.add_argument("--quantize-bits", type=int, default=8, choices=(4, 8), help="code width of --stage quantize")
    ap.add_argument("--quantize-unrotate", action="store_true",
                    help="--stage quantize: keys are rotated back from their positions first (position-free cache)")
    ap.add_argument("--attention-two-tiles", action="store_true",
                    help="run kvb_selective_attn with two tiles per CTA sharing K/V (the context's attention_two_tiles option)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    global ONE_PASS
    ONE_PASS = args.path == "one-pass"
    head_key = HEADLINE if args.workload == "all" else args.workload
    if args.requests > 0 and head_key != "cfg4":
        ap.error("--requests applies to --workload cfg4")
    wl = named_workload(head_key, args)
    if args.impl == "reference":
        run_reference(args, head_key, wl)
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

    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    run = Runner(args, B, dist, rank, world, local, sampler)

    if args.stage != "path":
        line = run.measure_stage(args.stage, head_key, wl)
        sampler.stop()
        if rank == 0:
            print(json.dumps(line))
        if dist:
            dist.destroy_process_group()
        return

    head = run.measure(head_key, wl, headline=True)
    per_config = {}
    if args.workload == "all" and world == 1:  # the other configurations, same build, same process
        for key in ("cfg1", "cfg2", "cfg3"):
            r = run.measure(key, named_workload(key, args), headline=False)
            per_config[key] = {k: r[k] for k in ("workload", "ms_per_step", "value", "tokens_per_step", "regions", "stages", "gpu_launches", "clocks", "l2")}
    sampler.stop()

    sh = wl.shape
    line = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if sh.kv_dtype == "bf16" else "fp16", "data": "synthetic",
        "config": config_dict(wl, PATH_NAMES[ONE_PASS] if head_key != "cfg3" else "kvb_selective_attn", args.meta_fp16, world, args.replicas or REPLICAS[head_key], args.attention_pairs),
        "resident": head["l2"],
        "roofline": head["roofline"], "stages": head["stages"], "regions": head["regions"],
        "instrumented_ms_per_step": head["instrumented_ms_per_step"], "gpu_launches": head["gpu_launches"],
        "clocks": head["clocks"], "wall_s_timed": head["wall_s_timed"],
    }
    for k in ("e2e", "cpu_baseline"):
        if k in head:
            line[k] = head[k]
    if per_config:
        line["per_config"] = per_config
    if rank == 0:
        print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
