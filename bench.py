#!/usr/bin/env python
"""Benchmark of the AudioKV eviction pass: one step = one audiokv_evict call over the whole
attention stack of the Qwen2.5-Omni-7B-shaped workload (28 layers, L = 8192).

Prints ONE JSON line (rank 0). `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2604_06694_b200 import workloads as wl  # noqa: E402

METRIC = "evict_pass_us_per_layer"
UNIT = "us/layer"
NOMINAL_HBM_GBS = 8000.0


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


KERNEL_SOURCES = {"score_umma_stats": "score_umma.cu", "score_umma_colsum": "score_umma.cu",
                  "score_simt_stats": "score_simt.cu", "score_simt_colsum": "score_simt.cu", "sss_select": "sss.cu",
                  "sss": "sss.cu", "select": "select_gather.cu", "gather": "select_gather.cu"}


def source_digest(kernel: str):
    """First 12 hex digits of the SHA-1 of the kernel's source file: a traffic figure counts only for the source it
    was captured on."""
    import hashlib
    f = KERNEL_SOURCES.get(kernel)
    path = os.path.join(ROOT, "paper_2604_06694_b200", "csrc", f) if f else None
    if not path or not os.path.exists(path):
        return None
    with open(path, "rb") as fh:
        return hashlib.sha1(fh.read()).hexdigest()[:12]


def captured_traffic(kernel: str, workload: str, layers: int):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum of one profiler capture) recorded for this
    kernel, workload and layer count in the traffic table beside the profiler summaries; None when there is no record
    or the kernel's source has changed since. Lines: kernel workload layers bytes source-digest."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    digest = source_digest(kernel)
    with open(path) as fh:
        for line in fh:
            f = line.split()
            if len(f) >= 5 and not line.startswith("#") and f[0] == kernel and f[1] == workload and int(f[2]) == layers \
                    and f[4] == digest:
                return int(f[3])
    return None


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled every 200 ms while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            pass

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def contract_bytes_per_layer(spec, w):
    """K read once plus kept K and V written, all requests of the batch, per layer: the least traffic one layer of
    the pass can have."""
    e = 4 if spec.dtype == "f32" else 2
    NL = w.full_layers or spec.n_layers
    row = spec.head_dim * e
    kept_rows_per_layer = int(w.total_budget.sum()) / NL
    return int(w.sum_L * spec.n_kv_heads * row + 2 * kept_rows_per_layer * row)


def kernel_algorithmic_bytes(name, spec, w):
    """Bytes each kernel must move per launch at this workload (what it reads once plus what it writes)."""
    e = 4 if spec.dtype == "f32" else 2
    NL, Hkv, d, W, Hq = spec.n_layers, spec.n_kv_heads, spec.head_dim, spec.window, spec.n_q_heads
    sumL = w.sum_L
    k_bytes = NL * Hkv * sumL * d * e
    q_bytes = len(spec.seq_lens) * NL * W * Hq * d * e
    score_bytes = 4 * NL * Hkv * (sumL - W * len(spec.seq_lens))
    kept_rows = int(w.total_budget.sum()) * NL // (w.full_layers or NL)
    if name.startswith("score") and "stats" in name:
        return k_bytes + q_bytes
    if name.startswith("score"):
        return k_bytes + q_bytes + score_bytes
    if name == "sss":
        return 2 * score_bytes
    if name in ("select", "sss_select"):
        return score_bytes + 4 * kept_rows
    if name == "gather":
        return kept_rows * (4 + 4 * d * e)           # index + K,V row read + K,V row written
    return 0


def kernel_algorithmic_exps(name, spec, w):
    """exp2 evaluations the softmax of each scoring sweep needs per launch: one per (window row, query head,
    visible key) in the statistics sweep, one per (window row, query head, prefix key) in the column-sum sweep."""
    NL, W, Hq = spec.n_layers, spec.window, spec.n_q_heads
    n = 0
    for L in spec.seq_lens:
        P = L - W
        if "stats" in name:
            n += NL * Hq * sum(P + i + 1 for i in range(W))
        else:
            n += NL * Hq * W * P
    return n


def kernel_algorithmic_flops(name, spec, w):
    """Multiply-adds x 2 of the Q K^T contraction one scoring sweep needs (every window row against every key)."""
    return 2 * spec.n_layers * spec.window * spec.n_q_heads * w.sum_L * spec.head_dim


# exp2 per clock and SM when both pipes that can produce them are full: the special-function unit gives 4 per clock
# and scheduler; the FMA pipe (32 lanes per clock and scheduler) spends 2 lane-operations on an exponential that goes
# to the special-function unit (scale-and-shift, accumulate) and 9 on one it evaluates itself (range reduction 3,
# cubic 3, exponent 1, scale-and-shift and accumulate 2): 4 + (32 - 8) / 9 = 6.67 per scheduler, four schedulers.
EXP2_PER_CLK_SM = 4 * (4 + (32 - 2 * 4) / 9.0)


def kernel_roofline(name, ms, spec, w, peaks, sm_max_mhz, sm_mhz, n_sm):
    """Roofline entry of one kernel: the scoring sweeps are bound by the exponentials (special-function unit plus
    the share the FMA pipe can take, at the maximum SM clock), everything else by HBM (measured copy bandwidth)."""
    nbytes = kernel_algorithmic_bytes(name, spec, w)
    traffic = captured_traffic(name, spec.name, spec.n_layers)
    hbm = nbytes / (ms * 1e-3) / 1e9 if ms > 0 else 0.0
    if name.startswith("score_umma"):
        peak = n_sm * EXP2_PER_CLK_SM * (sm_max_mhz or 1965.0) * 1e6 / 1e9      # Gexp2/s
        n_exp = kernel_algorithmic_exps(name, spec, w)
        ach = n_exp / (ms * 1e-3) / 1e9
        tflops = kernel_algorithmic_flops(name, spec, w) / (ms * 1e-3) / 1e12
        return {"kernel": name, "bound": "alu", "achieved": round(ach, 1), "peak": round(peak, 1), "unit": "Gexp2/s",
                "frac": round(ach / peak, 4),
                "frac_at_sampled_clock": round(ach / (peak * sm_mhz / sm_max_mhz), 4) if sm_mhz and sm_max_mhz else None,
                "peak_kind": f"{n_sm} SMs x {EXP2_PER_CLK_SM:.2f} exp2/clk (special-function unit + FMA-pipe share) x max SM clock",
                "algorithmic_exp2": n_exp, "algorithmic_bytes": nbytes,
                "hbm_gbs": round(hbm, 1), "hbm_frac_of_measured": round(hbm / peaks["hbm_gbs"], 4),
                "tensor_tflops": round(tflops, 1),
                "tensor_frac_of_measured_sustained": round(tflops / peaks["bf16_tflops_sustained"], 4),
                "traffic": traffic}
    return {"kernel": name, "bound": "hbm", "achieved": round(hbm, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": round(hbm / peaks["hbm_gbs"], 4), "algorithmic_bytes": nbytes,
            "traffic": traffic}


def rank_seed(rank: int) -> int:
    """Every rank evicts a request of its own (weak scaling, no exchange step): rank r draws the workload with seed r."""
    return rank


def max_over_ranks(x: float, world: int, device="cpu") -> float:
    """The slowest rank's time: all-reduce MAX over the default process group (identity when there is one rank)."""
    if world <= 1:
        return float(x)
    import torch.distributed as dist
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_us_per_layer(ms_step_max: float, n_layers: int, world: int) -> float:
    """All ranks run n_layers layers each in ms_step_max: microseconds per layer of the whole job."""
    return ms_step_max * 1e3 / (n_layers * world)


class Case:
    """One workload resident on the device, with its outputs and context, and the step that evicts it."""

    def __init__(self, B, w, local, over, sharded=False):
        self.B, self.w, self.spec, self.sharded = B, w, w.spec, sharded
        spec = w.spec
        over = dict(over)
        k_host, v_host = over.pop("_k_host", w.k), over.pop("_v_host", w.v)   # a paged pool instead of the plain cache
        self.prob = B.Problem.from_workload(w, **over)
        self.tb = [int(x) for x in w.total_budget]
        self.rows, self.TH = sum(self.tb), self.prob.total_heads
        es = w.torch_dtype()
        self.q, self.k, self.v = (w.as_torch(a).cuda() for a in (w.q, k_host, v_host))
        self.S = torch.from_numpy(w.head_scores).cuda()
        self.k_out = torch.empty((self.rows, spec.head_dim), dtype=es, device="cuda")
        self.v_out = torch.empty_like(self.k_out)
        self.kept = torch.empty(self.rows, dtype=torch.int32, device="cuda")
        self.budgets = torch.empty(self.TH, dtype=torch.int32, device="cuda")
        self.cu = torch.empty(self.TH + 1, dtype=torch.int32, device="cuda")
        ws_host = B.audiokv_workspace_bytes_host(self.prob, w.q.size, w.k.size, self.tb)
        self.ctx = B.Context(self.prob, device=local, workspace_bytes=ws_host)
        self.extra_launches_per_step = 0
        if sharded:
            # every step: the allocation over the whole stack (a second context planned for all layers; it touches no
            # K, V or Q), then steps 1, 2, 4 on this rank's layers with its slice of the budgets. With one request the
            # slice is a contiguous run of the table: a view, no copy.
            assert len(spec.seq_lens) == 1
            w_all = dataclasses.replace(w, spec=dataclasses.replace(spec, n_layers=w.full_layers))
            self.prob_all = B.Problem.from_workload(w_all, **over)
            self.ctx_all = B.Context(self.prob_all, device=local)
            TH_all = self.prob_all.total_heads
            self.budgets_all = torch.empty(TH_all, dtype=torch.int32, device="cuda")
            self.cu_all = torch.empty(TH_all + 1, dtype=torch.int32, device="cuda")
            self.mine = self.budgets_all[w.layer_begin * spec.n_kv_heads:(w.layer_begin + spec.n_layers) * spec.n_kv_heads]
            B.audiokv_allocate(self.ctx_all, self.prob_all, self.S, self.tb, self.budgets_all, self.cu_all)
            self.rows = int(self.mine.sum().item())
            self.k_out = torch.empty((self.rows, spec.head_dim), dtype=es, device="cuda")
            self.v_out = torch.empty_like(self.k_out)
            self.kept = torch.empty(self.rows, dtype=torch.int32, device="cuda")
            self.extra_launches_per_step = 1          # the allocation of the other context

    def step(self):
        B = self.B
        if self.sharded:
            B.audiokv_allocate(self.ctx_all, self.prob_all, self.S, self.tb, self.budgets_all, self.cu_all)
            B.audiokv_evict_budgeted(self.ctx, self.prob, self.q, self.k, self.v, self.mine, self.k_out, self.v_out,
                                     self.kept, self.cu)
        else:
            B.audiokv_evict(self.ctx, self.prob, self.q, self.k, self.v, self.S, self.tb, self.k_out, self.v_out,
                            self.kept, self.budgets, self.cu)

    def timed(self, steps, warmup, barrier, world, sampler=None):
        """ms per step (max over ranks) of `steps` steps after `warmup`, CUDA events on the launching stream."""
        for _ in range(max(warmup, 3)):
            self.step()
        barrier()
        stream = torch.cuda.current_stream()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n0 = self.ctx.launch_count()
        e0.record(stream)
        for _ in range(steps):
            self.step()
        e1.record(stream)
        barrier()
        launches = self.ctx.launch_count() - n0 + steps * self.extra_launches_per_step
        ms_total = e0.elapsed_time(e1)
        ms_step = max_over_ranks(ms_total, world, "cuda") / steps
        clocks = None
        if sampler:
            # nvidia-smi delivers a sample every 200 ms: when the timed region was shorter than about a second the
            # same step loop goes on (untimed) until the sampler has seen a second of this load
            t_load, extra = ms_total * 1e-3, 0
            while t_load < 1.2:
                for _ in range(200):
                    self.step()
                torch.cuda.synchronize()
                extra += 200
                t_load += 200 * ms_step * 1e-3
            clocks = sampler.stop()
            clocks["window"] = ("timed region" if extra == 0 else
                                f"timed region ({steps} steps) + {extra} more untimed steps of the same loop")
        assert self.ctx.last_device_status() == 0
        return ms_step, launches, clocks

    def per_kernel(self, steps):
        """Mean duration of each kernel of the step: the same loop with an event after every kernel."""
        self.ctx.profile_enable(True)
        acc = {}
        for _ in range(steps):
            self.step()
            for name, ms in self.ctx.profile_read():
                acc.setdefault(name, []).append(ms)
        self.ctx.profile_enable(False)
        torch.cuda.synchronize()
        return {n: statistics.mean(v) for n, v in acc.items()}


def run_cuda(args):
    from paper_2604_06694_b200 import binding as B
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    spec = wl.config(args.config)
    if args.window or args.keep:  # the keep x window sweep of the long-context configuration (not a bench line)
        spec = dataclasses.replace(spec, window=args.window or spec.window, keep=args.keep or spec.keep)
    sharded = args.shard == "layers"
    if sharded:
        # one request for the whole job, its layers dealt out over the ranks; no exchange step either: the budgets need
        # every head's score, which is a table of a few hundred floats that every rank holds
        n_full = args.layers or spec.n_layers
        w = wl.generate(spec, seed=0, layers=args.layers, layer_range=wl.layer_shard(n_full, world, rank))
    else:
        w = wl.generate(spec, seed=rank_seed(rank), layers=args.layers)   # every rank evicts its own request
    spec = w.spec
    over = dict(smooth_mode=args.smooth_mode, smooth_kappa=args.kappa, pool_kernel=args.pool_kernel)
    if args.page_size:
        # the same rows held in a pool of pages handed out in random order (the host-buffer leg has no paged form)
        k_host, v_host, table, n_pages, strides = wl.paged_pool(w, args.page_size, seed=rank_seed(rank))
        over.update(kv_strides=strides, kv_req_offset=None, page_size=args.page_size, n_pages=n_pages,
                    page_table=torch.from_numpy(table).cuda(), _k_host=k_host, _v_host=v_host)
        args.skip_e2e = True
    if sharded:
        args.skip_e2e = True

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    case = Case(B, w, local, over, sharded)
    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        time.sleep(0.3)                       # nvidia-smi needs a moment to start; the GPU idles meanwhile
    ms_step, launches, clocks = case.timed(args.steps, args.warmup, barrier, world, sampler)
    kern = case.per_kernel(min(args.steps, 200))
    score_path = case.ctx.last_score_path()

    e2e_ms, h2d, d2h = None, 0, 0
    if not args.skip_e2e:
        e2e_ms, h2d, d2h = run_e2e(B, case.ctx, case.prob, w, spec, case.tb, case.rows, case.TH, w.torch_dtype(),
                                   barrier, world, args)
    others = []
    if (world == 1 and args.config == 1 and not args.skip_other and not sharded and not args.layers and not args.page_size
            and not args.window and not args.keep):
        del case
        torch.cuda.empty_cache()
        for idx in (2, 3, 4):
            others.append(other_workload(B, idx, local, barrier, n_sm_of(local)))

    if rank != 0:
        if world > 1:
            torch.distributed.destroy_process_group()
        return
    job_layers = w.full_layers if sharded else spec.n_layers * world
    report(args, spec, w, world, ms_step, launches, kern, clocks, e2e_ms, h2d, d2h, job_layers, sharded, score_path,
           others, n_sm_of(local))
    if world > 1:
        torch.distributed.destroy_process_group()


def n_sm_of(local: int) -> int:
    return torch.cuda.get_device_properties(local).multi_processor_count


def workload_summary(spec, w, ms_step, job_layers, kern, score_path, peaks, n_sm, sm_max, sm_mhz):
    """The figures every workload is reported with: time per layer, contract bytes per second and their fractions,
    per-kernel durations and rooflines. Sums run over all requests of the batch."""
    cbytes = contract_bytes_per_layer(spec, w)
    hbm_gbs = cbytes * job_layers / (ms_step * 1e-3) / 1e9
    tot = sum(kern.values()) or 1.0
    roofs = [kernel_roofline(n, v, spec, w, peaks, sm_max, sm_mhz, n_sm) for n, v in kern.items()
             if n not in ("allocate", "budget_prefix")]
    return {
        "value": round(ms_step * 1e3 / job_layers, 4), "unit": UNIT, "ms_per_step": round(ms_step, 5),
        "tokens_heads_per_s": round(w.sum_L * spec.n_kv_heads * job_layers / (ms_step * 1e-3), 1),
        "hbm_gbs": round(hbm_gbs, 1),
        "hbm_frac_of_nominal_8tbs": round(hbm_gbs / NOMINAL_HBM_GBS, 4),
        "hbm_frac_of_measured": round(hbm_gbs / peaks["hbm_gbs"], 4),
        "contract_bytes_per_layer": cbytes,
        "score_path": score_path,
        "kernels_ms": {n: round(v, 5) for n, v in kern.items()},
        "kernel_share": {n: round(v / tot, 4) for n, v in kern.items()},
        "kernel_rooflines": roofs,
    }


def workload_config(spec, w, layers):
    lens = list(spec.seq_lens)
    return {"workload": spec.name, "layers": layers, "q_heads": spec.n_q_heads, "kv_heads": spec.n_kv_heads,
            "head_dim": spec.head_dim, "L": lens[0] if len(lens) == 1 else lens, "sum_L": w.sum_L,
            "requests_per_gpu": len(lens), "window": spec.window, "keep": spec.keep,
            "l2": "inputs larger than L2 (K+V of a step = %d MB)" % (2 * w.k.nbytes // 2**20)}


def other_workload(B, idx, local, barrier, n_sm, steps=20):
    """One of the other workloads of the metric's range (L = 16k and 32k, the ragged batch): the same measurement,
    fewer steps, no end-to-end or CPU leg."""
    w = wl.generate(wl.config(idx), seed=0)
    case = Case(B, w, local, {})
    ms_step, launches, _ = case.timed(steps, 3, barrier, 1)
    kern = case.per_kernel(10)
    peaks, _ = measured_peaks()
    out = {"config": workload_config(w.spec, w, w.spec.n_layers), "steps": steps, "dtype": w.spec.dtype,
           "gpu_launches": int(launches)}
    out.update(workload_summary(w.spec, w, ms_step, w.spec.n_layers, kern, case.ctx.last_score_path(), peaks, n_sm,
                                peaks.get("sm_max_mhz"), None))
    del case
    torch.cuda.empty_cache()
    return out


def run_e2e(B, ctx, prob, w, spec, tb, rows, TH, es, barrier, world, args):
    """End to end through the host-buffer entry point: pinned host inputs, results read back."""
    hq, hk, hv = (w.as_torch(a).pin_memory() for a in (w.q, w.k, w.v))
    hS = torch.from_numpy(w.head_scores).pin_memory()
    hko = torch.empty((rows, spec.head_dim), dtype=es).pin_memory()
    hvo = torch.empty_like(hko).pin_memory()
    hkept = torch.empty(rows, dtype=torch.int32).pin_memory()
    hb = torch.empty(TH, dtype=torch.int32).pin_memory()
    hcu = torch.empty(TH + 1, dtype=torch.int32).pin_memory()

    def step_host():
        B.audiokv_evict_host(ctx, prob, hq, hk, hv, hS, tb, hko, hvo, hkept, hb, hcu)

    step_host()
    barrier()
    # three groups of up to five calls, the median group: the host side of this leg (pinned-memory traffic, the link)
    # is shared with whatever else runs on the machine, and one disturbed group should not be the number
    n_e2e = max(1, min(args.steps, 5))
    groups = []
    for _ in range(3):
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            step_host()
        barrier()
        groups.append(max_over_ranks((time.perf_counter() - t0) * 1e3 / n_e2e, world, "cuda"))
    e2e_ms = sorted(groups)[1]
    # V is pinned: the gather fetches its kept rows from the host buffer itself, the other rows never cross the link
    h2d = sum(x.numel() * x.element_size() for x in (hq, hk, hS)) + hvo.numel() * hvo.element_size()
    d2h = sum(x.numel() * x.element_size() for x in (hko, hvo, hkept, hb, hcu))
    return e2e_ms, h2d, d2h


def report(args, spec, w, world, ms_step, launches, kern, clocks, e2e_ms, h2d, d2h, job_layers, sharded, score_path,
           others, n_sm):
    NL = spec.n_layers
    peaks, peak_kind = measured_peaks()
    sm_max = (clocks or {}).get("sm_max_mhz") or peaks.get("sm_max_mhz")
    sm_mhz = (clocks or {}).get("sm_mhz")
    summ = workload_summary(spec, w, ms_step, job_layers, kern, score_path, peaks, n_sm, sm_max, sm_mhz)
    roofs = {r["kernel"]: r for r in summ["kernel_rooflines"]}
    dom = max(roofs, key=lambda n: kern[n])          # the kernel that takes the largest share of the step
    roof = dict(roofs[dom])
    roof["peak_source"] = peak_kind
    cfg = workload_config(spec, w, job_layers if sharded else NL)
    cfg.update({"parallelism": (f"one request, layers sharded over {world} ranks ({NL} on rank 0), no collective"
                                if sharded else f"replicas x{world}, no collective"),
                "smooth_mode": args.smooth_mode, "page_size": args.page_size})
    line = {
        "metric": METRIC, "value": summ["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": summ["ms_per_step"], "higher_is_better": False,
        "scaling": "strong" if sharded else "weak", "vs_baseline": None, "dtype": spec.dtype, "data": "synthetic",
        "config": cfg,
    }
    for key in ("tokens_heads_per_s", "hbm_gbs", "hbm_frac_of_nominal_8tbs", "hbm_frac_of_measured",
                "contract_bytes_per_layer", "score_path"):
        line[key] = summ[key]
    line.update({
        "gpu_launches": int(launches),
        "kernels_ms": summ["kernels_ms"], "kernel_share": summ["kernel_share"],
        "roofline": roof,
        "kernel_rooflines": summ["kernel_rooflines"],
        "e2e": None if e2e_ms is None else
               {"value": round(e2e_ms * 1e3 / (NL * world), 3), "unit": UNIT, "ms_per_step": round(e2e_ms, 3),
                "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)},
        "clocks": clocks,
    })
    if others:
        line["other_workloads"] = others
    if not args.skip_cpu and world == 1:
        line["cpu_baseline"] = cpu_baseline(w, spec, budget_s=15.0)
    print(json.dumps(line), flush=True)


def oracle_pass(w, spec, n_layers):
    """The oracle's whole pass over the first n_layers layers of request 0; returns seconds."""
    import oracle
    L = spec.seq_lens[0]
    dims = (n_layers, spec.window, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, L)
    N = n_layers * spec.n_kv_heads
    Bt = int(np.floor(spec.keep * N * L))
    t0 = time.perf_counter()
    oracle.evict_request(w.q[0], w.k, w.v, oracle.BF16, dims, w.q_strides()[1:], w.kv_strides(),
                         1.0 / np.sqrt(spec.head_dim), w.head_scores[0, :n_layers], Bt, w.base,
                         float(np.float32(spec.rho)), float(np.float32(spec.alpha)), spec.transition_bins)
    return time.perf_counter() - t0


def cpu_baseline(w, spec, budget_s):
    """The oracle, as it stands, on the host cores: a bounded sample (the first layers) of the same workload."""
    cores = os.cpu_count() or 1
    t1 = oracle_pass(w, spec, 1)
    n = int(max(1, min(spec.n_layers, budget_s / max(t1, 1e-3))))
    t = oracle_pass(w, spec, n)
    return {"value": round(t * 1e6 / n, 1), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {n} of {spec.n_layers} layers of the same workload, all steps of the pass, OpenMP over heads"}


def run_reference(args):
    """The reference arm for this repository is the CPU oracle (there is no reference implementation to install)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    spec = wl.config(1)
    sample_layers = 4
    w = wl.generate(spec, seed=0, layers=sample_layers)
    for _ in range(max(args.warmup, 1)):
        oracle_pass(w, spec, sample_layers)
    ts, t_begin = [], time.perf_counter()
    for _ in range(args.steps):
        ts.append(oracle_pass(w, spec, sample_layers))
        if time.perf_counter() - t_begin > 120.0:     # a large --steps (the CUDA arm's default) stops after two minutes
            break
    sec = sum(ts) / len(ts)
    us_layer = sec * 1e6 / sample_layers
    cores = os.cpu_count() or 1
    sample = f"each step = the first {sample_layers} of {spec.n_layers} layers (all four steps of the pass)"
    line = {"impl": "reference", "metric": METRIC, "value": round(us_layer, 1), "unit": UNIT, "n_gpus": args.gpus,
            "steps": len(ts), "warmup": max(args.warmup, 1), "ms_per_step": round(sec * 1e3, 3),
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": spec.name, "layers": spec.n_layers, "L": spec.seq_lens[0], "window": spec.window,
                       "keep": spec.keep, "sample": sample},
            "cpu_baseline": {"value": round(us_layer, 1), "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": round(us_layer, 1), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--skip-cpu", action="store_true", help="leave out the CPU-oracle baseline (profiling runs)")
    ap.add_argument("--skip-e2e", action="store_true", help="leave out the host-buffer end-to-end leg (profiling runs)")
    ap.add_argument("--skip-other", action="store_true",
                    help="leave out the other workloads of the metric's range (L = 16k, 32k, ragged batch; 20 steps each)")
    ap.add_argument("--config", type=int, default=1,
                    help="workload index (1 = the benchmark workload; others are for exploration, not bench lines)")
    ap.add_argument("--smooth-mode", type=int, default=0,
                    help="0 = Spectral Score Smoothing (the benchmark); 1 fixed-fraction cut-off, 2 energy cut-off without "
                         "the mean, 3 average pooling, 4 max pooling (variants for ablation-style runs, not bench lines)")
    ap.add_argument("--kappa", type=float, default=0.5, help="cut-off fraction of --smooth-mode 1")
    ap.add_argument("--pool-kernel", type=int, default=7, help="window of --smooth-mode 3 and 4 (odd)")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "layers"],
                    help="N > 1: 'replicas' = one request per rank (weak scaling, the default); 'layers' = one request, "
                         "its layers dealt out over the ranks, budgets from one allocation over the whole stack (strong)")
    ap.add_argument("--page-size", type=int, default=0, choices=[0, 16, 32, 64, 128],
                    help="hold K and V in a pool of pages of this many tokens (0 = contiguous, the bench line)")
    ap.add_argument("--layers", type=int, default=None,
                    help="truncate the stack to its first LAYERS layers (small cases for profiler captures; not a bench line)")
    ap.add_argument("--window", type=int, default=None, help="observation window W instead of the configuration's (not a bench line)")
    ap.add_argument("--keep", type=float, default=None, help="retention ratio instead of the configuration's (not a bench line)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
