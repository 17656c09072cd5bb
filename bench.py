#!/usr/bin/env python
"""Throughput of the DART reduction step on synthetic LLaVA-NeXT-shaped batches.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload sweep_b256] [--pivots 8] [--keep 320] [--sweep]

One "step" is one pass of the whole reduction (scores, pivots, similarities, retention, packed
gather) over one batch.  Prints ONE JSON line on rank 0.  For N > 1 launch with torch.distributed.run:
every rank reduces its own batch (samples are independent; there is no collective on the data
path), the timed region is bracketed by a barrier and a device synchronise, and the time is the
maximum over ranks.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "vision_tokens_reduced_per_sec"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="sweep_b256")
    ap.add_argument("--pivots", type=int, default=None)
    ap.add_argument("--keep", type=int, default=None)
    ap.add_argument("--batch", type=int, default=None, help="override the workload's batch size")
    ap.add_argument("--sweep", action="store_true", help="also time every (pivots, keep) cell of the sweep")
    ap.add_argument("--path", type=int, default=0, help="0 auto, 1 staged, 2 fused (persistent sweep), 3 two passes (score pass + one tensor-core pass), 4 resident sweep, 5 split (resident for a share of the tiles, second read for the rest)")
    ap.add_argument("--tune", type=int, default=0, help="path 6: 16 * n1 + n2 ring depths")
    ap.add_argument("--split", type=int, default=0, help="path 5: k keeps tiles with index %% k == 0 on the chip, -k all others")
    ap.add_argument("--lag", type=int, default=0, help="fused path: extra tasks between a row's two sweeps")
    ap.add_argument("--retention", type=int, default=0, help="0 auto, 1 one kernel, 2 sorted lists + walks, 3 bands + turns, 4 bands and turns in one launch")
    ap.add_argument("--variants", action="store_true",
                    help="also time the variants: one threshold for all pivots, pivots given by the caller, KV-row gather")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


def pick_workload(args):
    from paper_2502_11494_b200 import workloads as W

    w = {c.name: c for c in W.CONFIGS + W.EXTRA}[args.workload]
    kw = {}
    if args.pivots:
        kw["n_pivot"] = args.pivots
    if args.keep:
        kw["n_keep"] = args.keep
    if args.batch:
        kw["B"] = args.batch
    return w.with_(**kw) if kw else w


def path_bytes_per_sample(w):
    """Algorithmic bytes of the whole step for one sample: the vision rows of the keys once, the kept
    hidden rows read and written, the packed indices and position ids."""
    return 2 * w.d * w.n_vis + 2 * (2 * w.d * w.S_out) + 12 * w.S_out


def kernel_bytes_per_launch(name, w, B):
    """Algorithmic bytes of one launch of a kernel, for B samples."""
    keys = 2 * w.d * w.n_vis * B
    return {
        "score": keys + 8 * w.n_vis * B,
        "sim": keys + 4 * w.n_pivot * w.n_vis * B,
        "sweep": keys,                       # fused scores + pivots + similarities: the keys count once
        "onepass": keys,                     # the caller's pivots: scores + similarities from one pass
        "resident": keys,                    # scores + pivots + similarities, rows held on the chip: one read
        "pair": keys,                        # paired sweeps: the second read of a row is meant to come from the L2
        "gather": 2 * (2 * w.d * w.S_out) * B,
        "pivot": 4 * w.n_vis * B,
        "retain": 4 * w.n_pivot * w.n_vis * B + 12 * w.S_out * B,
    }[name]


# DRAM traffic of one launch per sample (dram__bytes_read.sum + dram__bytes_write.sum), from ncu captures of each kernel
# on the sweep workload at batch 32; traffic is proportional to the batch (every sample is read and written
# independently), so a launch over B samples moves B times this.
NCU_TRAFFIC_PER_SAMPLE = {("sweep", 2880, 4096, 8): (1.508338e9 + 8.540928e6) / 32,
                          ("onepass", 2880, 4096, 8): (759.286272e6 + 5.440000e6) / 32,
                          ("resident", 2880, 4096, 8): (755.073536e6 + 6.136064e6) / 32}


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clock and throttle-reason samples taken while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower() == "active":
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    from paper_2502_11494_b200 import workloads as W

    oracle.build()
    w = pick_workload(args)
    total = args.steps + args.warmup
    per_step_budget = max(0.5, 150.0 / max(total, 1))
    k1, h1 = W.make_batch(w, device="cpu", samples=range(1))
    t0 = time.perf_counter()
    oracle.reduce(W.bits(h1), W.bits(k1), w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, want_dup=False)
    t1 = time.perf_counter() - t0
    n = int(max(1, min(w.B, per_step_budget / t1)))
    keys, hidden = W.make_batch(w, device="cpu", samples=range(n))
    kb, hb = W.bits(keys), W.bits(hidden)
    for _ in range(args.warmup):
        oracle.reduce(hb, kb, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, want_dup=False)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.reduce(hb, kb, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, want_dup=False)
    dt = time.perf_counter() - t0
    value = n * w.n_vis * args.steps / dt
    sample = "first %d of %d samples of %s per step" % (n, w.B, w.name)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, n),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def rank_samples(rank, B):
    """Weak scaling over independent samples: rank r reduces samples [r * B, (r + 1) * B) of the workload's
    seeded stream, so no two ranks hold the same sample and no data-path exchange is needed."""
    return range(rank * B, rank * B + B)


def max_over_ranks(value, device, dist_on):
    """The slowest rank's value (a job is as fast as its slowest rank)."""
    import torch
    import torch.distributed as dist

    t = torch.tensor([value], device=device, dtype=torch.float64)
    if dist_on:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_s(world, B, n_vis, steps, ms):
    """Whole-job throughput: the tokens all ranks reduced divided by the slowest rank's time."""
    return world * B * n_vis * steps / (ms * 1e-3)


L2_FLUSH_BYTES = 256 << 20      # written between timed steps when the inputs could stay in the 126 MB L2
L2_SAFE_INPUT_BYTES = 512 << 20  # inputs at least this large cannot be served from L2


def needs_flush(w, B):
    """True when the keys of one step could (partly) survive in L2 from one step to the next."""
    return 2 * B * w.S * w.d < L2_SAFE_INPUT_BYTES


def workload_config(w, B):
    return {"workload": w.name, "batch": B, "n_vis": w.n_vis, "seq_len": w.S, "d": w.d, "n_pivot": w.n_pivot,
            "n_keep": w.n_keep, "vis_offset": w.vis_offset,
            "l2": ("flushed between steps (%d MiB write), steps timed one by one" % (L2_FLUSH_BYTES >> 20)
                   if needs_flush(w, B) else "inputs larger than L2 (no flush needed)")}


def time_steps(ctx, dart, torch, w, keys, hidden, outs, steps, warmup, opts, dist_on, profile_steps=None):
    """Warm up, then time exactly `steps` reductions with CUDA events on the launching stream (no per-kernel events in
    that loop).  A second, profiled pass of `profile_steps` steps brackets every kernel launch with events: per-kernel
    durations and shares come from there.  Returns (total ms, per-step ms list, launches, profile dict)."""
    import torch.distributed as dist

    st = torch.cuda.current_stream()
    sp = ctypes.c_void_p(st.cuda_stream)
    P = lambda t: ctypes.c_void_p(t.data_ptr())  # noqa: E731

    def step():
        rc = dart.dart_reduce_ex(ctx.handle, P(hidden), P(keys), None, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep,
                                 P(outs[0]), P(outs[1]), P(outs[2]), opts, None, sp)
        if rc != 0:
            raise dart.DartError(rc, "dart_reduce_ex")

    flush = needs_flush(w, keys.shape[0])
    junk = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=keys.device) if flush else None

    def run(n):
        """n steps; small inputs: a buffer larger than L2 is written before every step and the steps are timed one by one"""
        if flush:
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
            for e0, e1 in evs:
                junk.fill_(1)
                e0.record(st)
                step()
                e1.record(st)
            torch.cuda.synchronize()
            per = [e0.elapsed_time(e1) for e0, e1 in evs]
            return sum(per), per
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
        evs[0].record(st)
        for i in range(n):
            step()
            evs[i + 1].record(st)
        torch.cuda.synchronize()
        return evs[0].elapsed_time(evs[n]), [evs[i].elapsed_time(evs[i + 1]) for i in range(n)]

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    dart.dart_profile_enable(ctx.handle, False)
    dart.dart_profile_read(ctx.handle)
    n0 = dart.dart_launch_count(ctx.handle)
    if dist_on:
        dist.barrier()
    torch.cuda.synchronize()
    ms, per = run(steps)
    if dist_on:
        dist.barrier()
    launches = dart.dart_launch_count(ctx.handle) - n0
    # profiled pass (same call, every launch bracketed by events on the same stream)
    dart.dart_profile_enable(ctx.handle, True)
    run(profile_steps if profile_steps else max(3, min(steps, 20)))
    dart.dart_profile_enable(ctx.handle, False)
    _, prof = dart.dart_profile_read(ctx.handle)
    if ctx.status() != 0:
        raise RuntimeError("device status word reports an error")
    return ms, per, launches, prof


def oracle_leg(w, keys, hidden, ref_idx, budget_s):
    """The CPU baseline: the oracle as it stands, single-threaded on one core (the stated baseline) and the same
    single-threaded code over samples on all host cores (context).  The samples it computes are also compared with the
    timed run's kept indices: exact-match rate and a histogram of the oracle's selection margins."""
    import math
    from concurrent.futures import ThreadPoolExecutor

    import numpy as np

    import oracle
    from paper_2502_11494_b200 import workloads as W

    oracle.build()
    B = keys.shape[0]
    cores = os.cpu_count() or 1
    kb, hb = W.bits(keys[:1]), W.bits(hidden[:1])
    t0 = time.perf_counter()
    oracle.reduce(hb, kb, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, want_dup=False, want_hidden=False)
    t1 = time.perf_counter() - t0
    n1 = int(max(1, min(B, (budget_s / 2) / max(t1, 1e-6))))
    nall = int(max(1, min(B, 256, cores * (budget_s / 2) / max(t1, 1e-6))))
    nb = max(n1, nall)
    kb, hb = W.bits(keys[:nb]), W.bits(hidden[:nb])   # only the samples the two timed passes touch go to the host
    t0 = time.perf_counter()
    oracle.reduce(hb[:n1], kb[:n1], w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, want_dup=False, want_hidden=False)
    dt1 = time.perf_counter() - t0

    def one(i):
        return oracle.reduce(hb[i:i + 1], kb[i:i + 1], w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, want_dup=False, want_hidden=False)

    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=cores) as pool:
        res = list(pool.map(one, range(nall)))
    dta = time.perf_counter() - t0
    ref = ref_idx[:nall].cpu().numpy()
    exact = sum(int(np.array_equal(ref[i], res[i].out_idx[0])) for i in range(nall))
    margins = np.array([float(r.margin[0]) for r in res])
    edges = [0.0, 1e-6, 1e-5, 1e-4, 1e-3, 1e-2, math.inf]
    hist = {("<%g" % edges[k + 1]) if k + 1 < len(edges) - 1 else ">=%g" % edges[k]: int(((margins >= edges[k]) & (margins < edges[k + 1])).sum())
            for k in range(len(edges) - 1)}
    return {
        "value": n1 * w.n_vis / dt1, "unit": UNIT, "cores": 1, "kind": "oracle",
        "sample": "first %d of %d samples of %s, one pass, %.1f s" % (n1, B, w.name, dt1),
        "all_cores": {"value": nall * w.n_vis / dta, "unit": UNIT, "cores": cores,
                      "sample": "first %d samples, one single-threaded oracle call per sample on %d host threads, %.1f s" % (nall, cores, dta)},
        "parity_on_sample": {"samples": nall, "identical_to_timed_run": exact, "exact_match_rate": exact / nall,
                             "above_margin_1e-3": int((margins > 1e-3).sum()), "margin_histogram": hist},
    }


def main():
    args = parse()
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist

    from paper_2502_11494_b200 import dart, workloads as W

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist_on = world > 1
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if dist_on:
        dist.init_process_group("nccl", device_id=dev)
    w = pick_workload(args)
    B = w.B
    # weak scaling: every rank reduces its own batch of B samples
    keys, hidden = W.make_batch(w, device=dev, samples=rank_samples(rank, B))
    flags = 0 if args.no_e2e else dart.DART_FLAG_HOST_STAGING
    ctx = dart.Dart(B, w.S, w.d, max(w.n_pivot, max(W.SWEEP_PIVOTS) if args.sweep else 0),
                    max(w.n_keep, max(W.SWEEP_KEEP) if args.sweep else 0), device=local, flags=flags)
    dart.dart_set_shape(ctx.handle, B, w.S)
    opts = dart.dart_opts(0, 0, args.path, 0, args.lag, 0, args.retention, resident_split=args.split, tune=args.tune)

    def alloc_outs(wl):
        return (torch.empty((B, wl.S_out, wl.d), dtype=torch.bfloat16, device=dev),
                torch.empty((B, wl.S_out), dtype=torch.int32, device=dev),
                torch.empty((B, wl.S_out), dtype=torch.int64, device=dev))

    outs = alloc_outs(w)
    sampler = ClockSampler(local)
    sampler.start()
    ms, per_step, launches, prof = time_steps(ctx, dart, torch, w, keys, hidden, outs, args.steps, args.warmup, opts, dist_on)
    clocks = sampler.stop()
    ref_idx = outs[1].clone()  # the timed run's kept indices (the variants below write into the same buffers)
    ms = max_over_ranks(ms, dev, dist_on)
    ms_per_step = ms / args.steps
    value = job_tokens_per_s(world, B, w.n_vis, args.steps, ms)

    peak, peak_src = measured_peak()
    # dominant kernel = the slot with the largest share of the timed region
    dom = max(prof, key=lambda k: prof[k][0]) if prof else None
    roofline = None
    if dom and prof[dom][1] > 0:
        avg_ms = prof[dom][0] / prof[dom][1]
        achieved = kernel_bytes_per_launch(dom, w, B) / (avg_ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak,
                    "traffic": (NCU_TRAFFIC_PER_SAMPLE[(dom, w.n_vis, w.d, w.n_pivot)] * B
                                if (dom, w.n_vis, w.d, w.n_pivot) in NCU_TRAFFIC_PER_SAMPLE and args.lag == 0 and args.tune == 0 else None),
                    "peak_source": peak_src + " copy bandwidth",
                    "avg_launch_ms": avg_ms, "timing": "CUDA events around every launch of a separate profiled pass on the launching stream",
                    "shares": {k: v[0] / max(sum(x[0] for x in prof.values()), 1e-9) for k, v in prof.items()}}
    path_gbs = path_bytes_per_sample(w) * B / (ms_per_step * 1e-3) / 1e9
    path_roof = {"algorithmic_bytes_per_step": path_bytes_per_sample(w) * B, "achieved": path_gbs, "unit": "GB/s",
                 "frac_of_measured_copy": path_gbs / peak, "frac_of_nominal_8TBs": path_gbs / 8000.0}

    sweep = None
    if args.sweep and rank == 0:
        sweep = []
        for (p, k) in W.sweep_cells():
            wc = w.with_(n_pivot=p, n_keep=k)
            o2 = alloc_outs(wc)
            ms2, _, _, _ = time_steps(ctx, dart, torch, wc, keys, hidden, o2, max(3, args.steps // 4), 2, opts, False, profile_steps=1)
            n2 = max(3, args.steps // 4)
            sweep.append({"n_pivot": p, "n_keep": k, "ms_per_step": ms2 / n2,
                          "tokens_per_s": B * wc.n_vis * n2 / (ms2 * 1e-3),
                          "path_frac_of_measured_copy": path_bytes_per_sample(wc) * B / (ms2 / n2 * 1e-3) / 1e9 / peak})
            del o2

    variants = None
    if args.variants and rank == 0:
        variants = {}
        n_v = max(3, args.steps // 4)
        # (a) retention with one threshold for all pivots
        o_g = dart.dart_opts(path=args.path, sweep_lag=args.lag, retention=args.retention, rule=dart.DART_RULE_GLOBAL)
        ms_g, _, _, prof_g = time_steps(ctx, dart, torch, w, keys, hidden, outs, n_v, 2, o_g, False, profile_steps=3)
        variants["one_threshold"] = {"ms_per_step": ms_g / n_v, "tokens_per_s": B * w.n_vis * n_v / (ms_g * 1e-3),
                                     "retain_ms": prof_g["retain"][0] / max(prof_g["retain"][1], 1)}
        # (a2) independent pivots (Eq. 10's union): variable-length packed outputs + cu_seqlens
        cu = torch.zeros(B + 1, dtype=torch.int32, device=dev)
        o_u = dart.dart_opts(path=args.path, sweep_lag=args.lag, retention=args.retention, rule=dart.DART_RULE_UNION,
                             cu_seqlens=cu.data_ptr())
        ms_u, _, _, prof_u = time_steps(ctx, dart, torch, w, keys, hidden, outs, n_v, 2, o_u, False, profile_steps=3)
        variants["independent_pivots"] = {"ms_per_step": ms_u / n_v, "tokens_per_s": B * w.n_vis * n_v / (ms_u * 1e-3),
                                          "retain_ms": prof_u["retain"][0] / max(prof_u["retain"][1], 1) * 3,  # three launches
                                          "mean_kept_vision_tokens": float(cu[-1].item()) / B - (w.S - w.n_vis)}
        # (b) pivots named by the caller (here: random distinct tokens): steps 3-5 only wait for the norms
        piv = torch.stack([torch.randperm(w.n_vis, device=dev)[:w.n_pivot] for _ in range(B)]).to(torch.int32).contiguous()
        o_p = dart.dart_opts(path=args.path, sweep_lag=args.lag, retention=args.retention, pivots_in=piv.data_ptr())
        ms_p, _, _, prof_p = time_steps(ctx, dart, torch, w, keys, hidden, outs, n_v, 2, o_p, False, profile_steps=3)
        variants["pivots_given"] = {"ms_per_step": ms_p / n_v, "tokens_per_s": B * w.n_vis * n_v / (ms_p * 1e-3),
                                    "path_frac_of_measured_copy": path_bytes_per_sample(w) * B / (ms_p / n_v * 1e-3) / 1e9 / peak}
        if prof_p.get("onepass", (0, 0))[1]:
            ms_o = prof_p["onepass"][0] / prof_p["onepass"][1]
            gbs_o = kernel_bytes_per_launch("onepass", w, B) / (ms_o * 1e-3) / 1e9
            tr = NCU_TRAFFIC_PER_SAMPLE.get(("onepass", w.n_vis, w.d, w.n_pivot))
            variants["pivots_given"]["onepass_kernel"] = {"ms_per_launch": ms_o, "achieved_GBps": gbs_o,
                                                          "frac_of_measured_copy": gbs_o / peak,
                                                          "traffic": tr * B if tr else None}
        # (b1) the caller's pivots drawn from the whole sample, text tokens included (indices relative to the vision block)
        piv_t = (torch.stack([torch.randperm(w.S, device=dev)[:w.n_pivot] for _ in range(B)]) - w.vis_offset).to(torch.int32).contiguous()
        o_t = dart.dart_opts(path=args.path, sweep_lag=args.lag, retention=args.retention, text_pivots=1, pivots_in=piv_t.data_ptr())
        ms_t, _, _, _ = time_steps(ctx, dart, torch, w, keys, hidden, outs, n_v, 2, o_t, False, profile_steps=1)
        variants["text_pivots"] = {"ms_per_step": ms_t / n_v, "tokens_per_s": B * w.n_vis * n_v / (ms_t * 1e-3),
                                   "path_frac_of_measured_copy": path_bytes_per_sample(w) * B / (ms_t / n_v * 1e-3) / 1e9 / peak}
        del piv_t
        # (b2) pivots ranked by the key rows, Eq. 7 on the hidden rows: keys once (scores), hidden once (one pass)
        o_h = dart.dart_opts(path=args.path, sweep_lag=args.lag, retention=args.retention, cosine_on_hidden=1)
        ms_h, _, _, prof_h = time_steps(ctx, dart, torch, w, keys, hidden, outs, n_v, 2, o_h, False, profile_steps=3)
        bytes_h = (path_bytes_per_sample(w) + 2 * w.d * w.n_vis) * B   # one more read of n_vis x d than the main method
        variants["cosine_on_hidden"] = {"ms_per_step": ms_h / n_v, "tokens_per_s": B * w.n_vis * n_v / (ms_h * 1e-3),
                                        "algorithmic_bytes_per_step": bytes_h,
                                        "path_frac_of_measured_copy": bytes_h / (ms_h / n_v * 1e-3) / 1e9 / peak,
                                        "kernel_ms": {k_: v_[0] / v_[1] for k_, v_ in prof_h.items() if v_[1]}}
        # (c) the key rows of the retained tokens, packed by the list of the last reduction (one KV tensor of one layer)
        packed = torch.empty_like(outs[0])
        st = torch.cuda.current_stream()
        P_ = lambda t: ctypes.c_void_p(t.data_ptr())  # noqa: E731
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for k_ in range(2 + n_v):
            if k_ == 2:
                e0.record(st)
            rc = dart.dart_gather_rows(P_(keys), P_(outs[1]), B, w.S, w.S_out, 2 * w.d, P_(packed), local,
                                       ctypes.c_void_p(st.cuda_stream))
            if rc != 0:
                raise dart.DartError(rc, "dart_gather_rows")
        e1.record(st)
        torch.cuda.synchronize()
        ms_k = e0.elapsed_time(e1) / n_v
        gbs = 2 * (2 * w.d * w.S_out) * B / (ms_k * 1e-3) / 1e9
        variants["kv_row_gather"] = {"ms_per_launch": ms_k, "achieved_GBps": gbs, "frac_of_measured_copy": gbs / peak}
        del packed, piv

    e2e = None
    if not args.no_e2e:
        # the same step through the host-buffer entry point: pinned inputs -> device -> pinned outputs
        import psutil

        need = 2 * keys.numel() * 2 + outs[0].numel() * 2
        Be = B
        while Be > 1 and need * Be // B * 2 > psutil.virtual_memory().available:
            Be //= 2
        hk = keys[:Be].cpu().pin_memory()
        hh = hidden[:Be].cpu().pin_memory()
        ho = (torch.empty((Be, w.S_out, w.d), dtype=torch.bfloat16).pin_memory(),
              torch.empty((Be, w.S_out), dtype=torch.int32).pin_memory(),
              torch.empty((Be, w.S_out), dtype=torch.int64).pin_memory())
        dart.dart_set_shape(ctx.handle, Be, w.S)
        P = lambda x: ctypes.c_void_p(x.data_ptr())  # noqa: E731
        n_e2e = 2

        def host_step():
            rc = dart.dart_reduce_host(ctx.handle, P(hh), P(hk), w.vis_offset, w.n_vis, w.n_pivot, w.n_keep,
                                       P(ho[0]), P(ho[1]), P(ho[2]))
            if rc != 0:
                raise dart.DartError(rc, "dart_reduce_host")

        host_step()
        if dist_on:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            host_step()
        dt = time.perf_counter() - t0
        dt = max_over_ranks(dt, dev, dist_on)
        ok = bool(torch.equal(ho[1], ref_idx[:Be].cpu())) if not args.sweep else None
        e2e = {"value": world * Be * w.n_vis * n_e2e / dt, "unit": UNIT,
               "h2d_bytes_per_step": int(hk.numel() * 2 + hh.numel() * 2),
               "d2h_bytes_per_step": int(sum(x.numel() * x.element_size() for x in ho)),
               "samples": Be, "steps": n_e2e, "ms_per_step": 1e3 * dt / n_e2e, "matches_device_run": ok}
        dart.dart_set_shape(ctx.handle, B, w.S)

    cpu = None
    if rank == 0 and not args.no_cpu_baseline:
        cpu = oracle_leg(w, keys, hidden, ref_idx, budget_s=20.0)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step,
            "ms_per_step_median": sorted(per_step)[len(per_step) // 2], "ms_per_step_best": min(per_step),
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16 in, f32 accumulate", "data": "synthetic",
            "config": workload_config(w, B), "roofline": roofline, "path_roofline": path_roof,
            "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
        }
        if sweep is not None:
            line["sweep"] = sweep
        if variants is not None:
            line["variants"] = variants
        print(json.dumps(line))
    ctx.close()
    if dist_on:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
