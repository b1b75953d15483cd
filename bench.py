"""Benchmark of the cached mixed-precision embedding training step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--impl ours|reference]

One "step" is mpe_forward + mpe_backward over one batch of the chosen
configuration (default: configuration 4, the largest one, 64 tables x 5M rows x
dim 128, packed INT4, 1% FP32 cache, LFU).  Inputs are seeded synthetic Zipf
streams generated on the device before the timed region (every batch is far
larger than L2).  Timing uses CUDA events on the stream the kernels are launched
on.  With N > 1 (torchrun) every rank trains its own shard of tables of the
same size (weak scaling, no data-path collective) and rank 0 reports the
aggregate.  Prints ONE JSON line.

--impl reference times the CPU oracle (oracle/) on the host cores on a bounded
sample of the same workload.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)
from paper_2010_11305_b200 import workloads as wl  # noqa: E402

METRIC = "embedding rows/sec per training step (fwd+bwd+cache) and % of 8 TB/s HBM"
NOMINAL_HBM_GBS = 8000.0
# What ncu showed for the heavy kernels on 8 of the 64 tables of configuration 4 (same shapes per table; DRAM traffic grows in
# proportion to the indices processed): dram__bytes_read.sum + dram__bytes_write.sum per index of the batch, and the
# limiter the counters point at.  The summaries under profiles/ give the commands and the counters.
KERNEL_EVIDENCE = {
    "update": {"dram_bytes_per_index": 112.7, "bound": "issue",
               "evidence": "80 % of the issue slots used, 317 warp instructions per distinct row; DRAM 29 %, L2 26 % of peak",
               "profile": "profiles/k_update_cfg4_8tables.md"},
    "pool": {"dram_bytes_per_index": 72.8, "bound": "latency",
             "evidence": "7.3 long-scoreboard stall cycles per issue at 46 % of the warp slots (64 registers); L1 50 %, DRAM 22 % of peak; 61 % of the sectors hit in L1",
             "profile": "profiles/k_pool_cfg4_8tables.md"},
    "hot_partial": {"dram_bytes_per_index": 20.9, "bound": "l2-latency",
                    "evidence": "gradient rows come from L2 (83 % hits, 36 % of its throughput), 11.2 long-scoreboard stall cycles per issue at 24 % of the warp slots (kept small on purpose: it runs beside other kernels)",
                    "profile": "profiles/k_hot_partial_cfg4_8tables.md"},
    # on the small case a pass of the sort is L2 resident, so its DRAM traffic does not scale to the full size: none given
    "sort_scatter": {"dram_bytes_per_index": None, "bound": "latency",
                     "evidence": "short scoreboard 6.1 (ranking through shared-memory counters), long scoreboard 5.6 (tile load, look-back) and barrier 2.6 stall cycles per issue; 35 % of the issue slots; DRAM 14 %, L2 24 % of peak",
                     "profile": "profiles/k_sort_scatter_cfg4_9tables.md"},
    "broadcast": {"dram_bytes_per_index": 14.1, "bound": "l2",
                  "evidence": "64 % of the L2 throughput (4-byte scatters and gathers inside a table's window), 80 long-scoreboard and 13.6 lg_throttle stall cycles per issue",
                  "profile": "profiles/k_broadcast_cfg4_8tables.md"},
    "priority": {"dram_bytes_per_index": 16.2, "bound": "dram-latency",
                 "evidence": "one random read-modify-write of a counter per distinct row: 30 long-scoreboard stall cycles per issue, 13 % of the issue slots",
                 "profile": "profiles/small_kernels_cfg4_8tables.md"},
    "policy": {"dram_bytes_per_index": 6.3, "bound": "latency",
               "evidence": "8.8 long-scoreboard stall cycles per issue, 47 % of the issue slots",
               "profile": "profiles/small_kernels_cfg4_8tables.md"},
}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, gpu_index):
        self.q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
                  "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        self.gpu = gpu_index
        self.proc = None
        self.lines = []            # (arrival time, text)
        self.t_begin = self.t_end = None

    def begin(self):
        self.t_begin = time.perf_counter()

    def end(self):
        self.t_end = time.perf_counter()

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.q}", "--format=csv,noheader,nounits",
                                          "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line.strip()))

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        # the samples taken while the timed steps ran (a sample describes the interval before it arrives); all of them
        # if the region was too short to catch one
        inside = [l for t, l in self.lines if self.t_begin is not None and self.t_end is not None and self.t_begin <= t <= self.t_end + 0.03]
        for l in (inside or [l for _, l in self.lines]):
            f = [x.strip() for x in l.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); smax.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "during_timed_steps": bool(inside), "reasons": sorted(reasons)}


def describe(cfg):
    pol = "LFU" if cfg.policy == wl.LFU else "LRU"
    opt = "row-wise Adagrad" if cfg.optimizer == wl.ROWWISE_ADAGRAD else "SGD"
    return (f"{cfg.name}: {cfg.num_tables} tables x {max(cfg.num_rows):,} rows x dim {cfg.dim}, {"FP16" if cfg.bits == 16 else "INT%d row-wise" % cfg.bits}, "
            f"cache {cfg.cache_fraction:g} x rows, {cfg.ways or 32}-way {pol}, batch {cfg.batch}, bags {cfg.bag}, {opt}")


def byte_model(cfg, L, U, U_hit, occ_hit, admissions, evictions, hot_occ, passes_main, passes_cand):
    """Algorithmic bytes of one step, counted both ways.

    per access  -- what the METHOD moves if every access goes to memory (the paper's effective-bandwidth numerator,
                   Section 5.2): per index 4 B of id plus the fetched row (FP32 row on a hit, codes + scale + bias on a
                   miss), the pooled output, one gradient row per index, per distinct row a read and a write of its home
                   (FP32 row or quantized row), the priority update, the optimizer state, evictions (FP32 read +
                   quantized write), admissions (FP32 write), and the de-duplication minimum 8 L + 4 U;
    compulsory  -- the same with every distinct byte counted once per pass: rows per DISTINCT row instead of per index,
                   the gradient tensor once; a lower bound of the DRAM traffic.

    Returns (per_access_step, compulsory_step, per_kernel) with per_kernel[name] = (per-access bytes, compulsory bytes,
    basis).  The per-kernel figures hold the method's bytes only (none of this implementation's bookkeeping arrays);
    kernels that are bookkeeping of this implementation and nothing else (the sort passes, the scatter of the probe
    results) are given the bytes their own algorithm has to move, and say so in `basis`.
    """
    d, T, B = cfg.dim, cfg.num_tables, cfg.batch
    rb = d * cfg.bits // 8 + (0 if cfg.bits == 16 else 8)      # codes + FP32 scale + FP32 bias (none for an FP16 table)
    fb = 4 * d
    occ_miss, U_miss = L - occ_hit, U - U_hit
    out_bytes = 4 * B * T * d
    pv = (8 * U) if cfg.policy == wl.LFU else (4 * U_hit)
    opt = (8 * U) if cfg.optimizer == wl.ROWWISE_ADAGRAD else 0
    rows_rw = U_hit * 2 * fb + (U_miss - admissions) * 2 * rb + admissions * (rb + fb) + evictions * (fb + rb)
    fwd = 4 * L + occ_hit * fb + occ_miss * rb + out_bytes
    bwd = L * fb + rows_rw + pv + opt
    dedup = 8 * L + 4 * U
    per_access = fwd + bwd + dedup
    compulsory = (4 * L + U_hit * fb + U_miss * rb + out_bytes) + (out_bytes + rows_rw + pv + opt) + dedup
    cold_occ = L - hot_occ
    m = {}
    m["pool"] = (fwd, 4 * L + U_hit * fb + U_miss * rb + out_bytes, "method")
    m["update"] = (cold_occ * fb + rows_rw + opt, min(cold_occ * fb, out_bytes) + rows_rw + opt, "method")
    m["hot_partial"] = (hot_occ * fb, min(hot_occ * fb, out_bytes), "method")
    m["priority"] = (pv, pv, "method")
    m["probe"] = (4 * cfg.ways * U, 4 * cfg.ways * U, "method (tag reads)")
    m["policy"] = (U_miss * (4 if cfg.policy == wl.LFU else 0) + admissions * 8 * cfg.ways,) * 2 + ("method (priority values of candidates and sets)",)
    sort_rw = passes_main * 16 * L + passes_cand * 16 * U
    m["sort_scatter"] = (sort_rw, sort_rw, "radix-sort pass: key + payload read and written")
    m["sort_digits"] = (4 * L + 8 * U,) * 2 + ("radix sort: the keys read once, ahead of the passes",)
    m["make_keys"] = (4 * L + 4 * T * B, 4 * L + 4 * T * B, "indices and offsets read")
    m["unique"] = (4 * L + 4 * U, 4 * L + 4 * U, "sorted keys read, distinct rows written")
    m["unique_count"] = (4 * L, 4 * L, "sorted keys read")
    m["unique_write"] = (4 * L + 4 * U, 4 * L + 4 * U, "sorted keys read, distinct rows written")
    m["broadcast"] = (8 * L, 8 * L, "bookkeeping: per-index slot and sample id written")
    return per_access, compulsory, m


def shard_config(cfg, rank):
    """Table-wise sharding without a data-path collective: every rank trains its own set of tables of the
    configuration's shapes (its own seed, hence its own rows and index streams): weak scaling."""
    cfg.seed = cfg.seed + 7919 * rank
    return cfg


def aggregate(times, rows, world, device):
    """Whole-job figures from per-rank ones: the slowest rank's times (MAX) and everybody's rows (SUM)."""
    if world <= 1:
        return [float(x) for x in times], [float(x) for x in rows]
    t = torch.tensor(times, dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    r = torch.tensor(rows, dtype=torch.float64, device=device)
    torch.distributed.all_reduce(r, op=torch.distributed.ReduceOp.SUM)
    return [float(x) for x in t], [float(x) for x in r]


def link_rate(dev, up_bytes, down_bytes):
    """Host link rate in this run: pinned copies of one step's sizes, timed with CUDA events: each direction alone, then
    both at once on two streams (what consecutive steps do when their uploads and downloads overlap)."""
    nu, nd = max(int(up_bytes) // 4, 1), max(int(down_bytes) // 4, 1)
    h_up, d_up = torch.empty(nu, dtype=torch.float32).pin_memory(), torch.empty(nu, dtype=torch.float32, device=dev)
    h_dn, d_dn = torch.empty(nd, dtype=torch.float32).pin_memory(), torch.empty(nd, dtype=torch.float32, device=dev)
    s_up, s_dn = torch.cuda.Stream(dev), torch.cuda.Stream(dev)

    def timed(up, down):
        best = None
        for _ in range(3):
            torch.cuda.synchronize(dev)
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            if up:
                with torch.cuda.stream(s_up):
                    ev[0].record(); d_up.copy_(h_up, non_blocking=True); ev[1].record()
            if down:
                with torch.cuda.stream(s_dn):
                    ev[2].record(); h_dn.copy_(d_dn, non_blocking=True); ev[3].record()
            torch.cuda.synchronize(dev)
            t = (ev[0].elapsed_time(ev[1]) if up else 0.0, ev[2].elapsed_time(ev[3]) if down else 0.0)
            best = t if best is None or max(t) < max(best) else best
        return best

    up_ms, dn_ms = timed(True, False)[0], timed(False, True)[1]
    both = timed(True, True)
    return {"h2d_ms": up_ms, "h2d_gbs": nu * 4 / up_ms / 1e6, "d2h_ms": dn_ms, "d2h_gbs": nd * 4 / dn_ms / 1e6,
            "both_at_once": {"h2d_ms": both[0], "h2d_gbs": nu * 4 / both[0] / 1e6, "d2h_ms": both[1], "d2h_gbs": nd * 4 / both[1] / 1e6}}


def kernel_roofline(name, tms, n, K, L, model, peak, peak_kind, evidence_ok, step_ms):
    """One kernel's record: per-access and compulsory bytes per launch over its CUDA-event time, and, where an ncu
    capture exists for this workload, its DRAM traffic and the limiter the counters showed."""
    per_launch_ms = tms / n
    lps = max(n / K, 1e-9)
    pa, comp, basis = model.get(name, (0.0, 0.0, "not modelled"))
    pa, comp = pa / lps, comp / lps
    ev = KERNEL_EVIDENCE.get(name) if evidence_ok else None
    traffic = ev["dram_bytes_per_index"] * L / lps if ev and ev["dram_bytes_per_index"] is not None else None
    sec = per_launch_ms * 1e-3
    achieved = pa / sec / 1e9 if sec > 0 else 0.0
    return {"kernel": name, "bound": ev["bound"] if ev else "unprofiled", "achieved": achieved, "peak": peak, "peak_kind": peak_kind,
            "unit": "GB/s", "frac": achieved / peak, "basis": "per-access bytes of the method / CUDA-event time; " + basis,
            "traffic": traffic, "dram_gbs": traffic / sec / 1e9 if traffic else None,
            "dram_frac": traffic / sec / 1e9 / peak if traffic else None,
            "bytes_per_launch": pa, "compulsory_bytes_per_launch": comp, "compulsory_frac": comp / sec / 1e9 / peak if sec > 0 else None,
            "ms_per_launch": per_launch_ms, "launches_per_step": n / K, "share_of_step": tms / K / step_ms,
            "evidence": ev["evidence"] if ev else None, "profile": ev["profile"] if ev else None}


def run_ours(args, cfg, rank, world, local_rank):
    from paper_2010_11305_b200 import binding as mpe
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    cfg = shard_config(cfg, rank)
    stream_gen = wl.Stream(cfg, dev)
    h = mpe.Mpe(cfg.num_rows, cfg.dim, cfg.bits, cfg.cache_fraction, cfg.ways, cfg.policy, cfg.optimizer, cfg.eps,
                cfg.init_lo, cfg.init_hi, cfg.seed, local_rank)
    n_e2e = min(args.steps, args.e2e_steps)
    total_steps = args.warmup + args.steps + n_e2e
    batches = [stream_gen.batch(s) for s in range(1, total_steps + 1)]
    maxL = max(b[0].numel() for b in batches)
    h.reserve(cfg.batch, maxL)
    out = torch.empty(cfg.batch, cfg.num_tables * cfg.dim, dtype=torch.float32, device=dev)
    # The step runs on a stream of higher priority than the one the next batch is prepared on (and than the library's own
    # second stream): when both have blocks ready, the step's kernels get the SMs first and the others fill the gaps.
    torch.cuda.synchronize(dev)
    torch.cuda.set_stream(torch.cuda.Stream(dev, priority=-1))
    cs = torch.cuda.current_stream(dev)
    sp = cs.cuda_stream

    counter = [0]       # the step number: strictly increasing over the handle's life

    # The next batch is sorted and de-duplicated on a second stream while the current step runs (mpe_prepare): that
    # part of a step needs the indices only.  Every timed step prepares its successor, so the work of K batches is
    # inside the region that times K steps.
    side = torch.cuda.Stream(dev)
    ahead = not args.no_prepare
    use_prepare = [ahead]

    def step(i):
        idx, off, grad = batches[i]
        counter[0] += 1
        h.forward(idx, off, cfg.batch, out, sp)
        if use_prepare[0] and i + 1 < len(batches):
            h.prepare(batches[i + 1][0], batches[i + 1][1], cfg.batch, side.cuda_stream)
        h.backward(grad, cfg.lr, counter[0])

    # Small steps are replayed from CUDA graphs (which per-kernel event records would break up) and large steps run
    # beside the next batch's preparation (which makes a kernel's bracketing events include its neighbours): the timed
    # region runs without the records, and the per-kernel times come from a second pass over the same batches, launched
    # plainly and without the preparation.
    graph_sized = maxL <= (4 << 20)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize(dev)

    for i in range(args.warmup):
        step(i)
    barrier()
    stats0 = np.sum([h.stats(t) for t in range(cfg.num_tables)], axis=0).astype(np.int64)
    launches0 = h.kernel_launches()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    barrier()
    K = args.steps
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]      # one record between every two steps
    sampler.begin()
    marks[0].record(cs)
    for j, i in enumerate(range(args.warmup, args.warmup + K)):
        step(i)
        marks[j + 1].record(cs)
    barrier()
    sampler.end()
    ms = marks[0].elapsed_time(marks[K])
    per_step_ms = [marks[j].elapsed_time(marks[j + 1]) for j in range(K)]
    clocks = sampler.stop()
    launches = h.kernel_launches() - launches0
    stats1 = np.sum([h.stats(t) for t in range(cfg.num_tables)], axis=0).astype(np.int64)
    code, detail = h.last_error()
    assert code == 0, f"device error {code} ({detail})"
    ds = stats1 - stats0
    L, occ_hit, U, U_hit, adm, evi = (ds[i] / K for i in (0, 1, 2, 3, 4, 5))
    hot_rows, hot_occ = float(h.step_info()[3]), float(h.step_info()[4])      # of the last timed step

    # End to end through the host-buffer entry point: pinned host inputs, H2D + step + D2H inside the timed region.
    # The steps are submitted back to back (mpe_step_host_submit) and waited for once, so the upload of one step runs
    # while the previous one computes; a second figure times the same steps one at a time (mpe_step_host).
    h_batches = []
    for i in range(args.warmup + args.steps, total_steps):
        idx, off, grad = batches[i]
        h_batches.append((idx.cpu().pin_memory(), off.cpu().pin_memory(), grad.cpu().pin_memory()))
    h_outs = [torch.empty(cfg.batch, cfg.num_tables * cfg.dim, dtype=torch.float32).pin_memory() for _ in range(min(2, max(n_e2e, 1)))]
    h2d = float(np.mean([(a.numel() + b.numel() + c.numel()) * 4 for a, b, c in h_batches])) if h_batches else 0.0
    d2h = float(h_outs[0].numel() * 4)
    e2e_rows, e2e_s, e2e_serial_s = 0, 0.0, 0.0
    link = None
    if h_batches:
        link = link_rate(dev, h2d, d2h)
        counter[0] += 1
        h.step_host(h_batches[0][0], h_batches[0][1], cfg.batch, h_batches[0][2], h_outs[0], cfg.lr, counter[0])   # sizes the staging buffers
        barrier()
        t0 = time.perf_counter()
        for j, (idx, off, grad) in enumerate(h_batches):
            counter[0] += 1
            h.step_host_submit(idx, off, cfg.batch, grad, h_outs[j % len(h_outs)], cfg.lr, counter[0])
            e2e_rows += idx.numel()
        h.step_host_wait()
        torch.cuda.synchronize(dev)
        e2e_s = time.perf_counter() - t0
        barrier()
        t0 = time.perf_counter()
        for j, (idx, off, grad) in enumerate(h_batches):
            counter[0] += 1
            h.step_host(idx, off, cfg.batch, grad, h_outs[0], cfg.lr, counter[0])
        torch.cuda.synchronize(dev)
        e2e_serial_s = time.perf_counter() - t0
    h.profile(True)
    use_prepare[0] = False
    for i in range(args.warmup, args.warmup + args.steps):
        step(i)
    prof = h.profile_read()
    h.profile(False)
    use_prepare[0] = ahead

    # aggregate over ranks: total rows / max time
    (ms, e2e_s, e2e_serial_s), (rows_timed, e2e_rows) = aggregate([ms, e2e_s, e2e_serial_s], [float(ds[0]), float(e2e_rows)], world, dev)
    if rank != 0:
        return None

    passes_main = (max(cfg.num_rows).bit_length() + 7) // 8
    max_sets = max(h.cache_geometry(t)[0] for t in range(cfg.num_tables))
    passes_cand = (max(max_sets, 1).bit_length() + 7) // 8 if max_sets else 0
    per_access, compulsory, model = byte_model(cfg, L, U, U_hit, occ_hit, adm, evi, hot_occ, passes_main, passes_cand)
    per_access, compulsory = float(per_access), float(compulsory)
    ms_step = ms / K
    ms_median = float(np.median(per_step_ms))
    peak, peak_kind = measured_peaks()
    # the ncu figures belong to configuration 4 as it is defined (INT4, LFU): variants and other configurations have none
    evidence_ok = args.config == 4 and args.bits is None and args.policy is None
    ranked = sorted(prof.items(), key=lambda kv: -kv[1][0])
    recs = [kernel_roofline(name, tms, n, K, L, model, peak, peak_kind, evidence_ok, ms_step) for name, (tms, n) in ranked[:5]]
    sec = ms_step * 1e-3
    result = {
        "metric": METRIC, "value": rows_timed / (ms * 1e-3), "unit": "rows/s", "n_gpus": world, "steps": K,
        "warmup": args.warmup, "ms_per_step": ms_step, "ms_per_step_median": ms_median, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": describe(cfg), "l2": "inputs larger than L2; a new batch every step",
                   "launch": ("CUDA graph replay" if graph_sized else "plain launches") + "; per-kernel times from a second, plainly launched pass without the preparation",
                   "next_batch": "sorted ahead on a second stream of lower priority (mpe_prepare) while the current step runs" if ahead and not graph_sized else "not prepared ahead",
                   "sharding": "each rank trains its own tables (no data-path collective)" if world > 1 else "one GPU"},
        "clocks": clocks,
        "e2e": {"value": e2e_rows / e2e_s if e2e_s > 0 else None, "unit": "rows/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": len(h_batches), "ms_per_step": 1e3 * e2e_s / max(len(h_batches), 1),
                "mode": "steps submitted back to back through mpe_step_host_submit, one wait at the end (uploads, kernels and downloads of neighbouring steps overlap)",
                "one_step_at_a_time": {"value": e2e_rows / e2e_serial_s if e2e_serial_s > 0 else None,
                                       "ms_per_step": 1e3 * e2e_serial_s / max(len(h_batches), 1)},
                "link": link,
                "link_bound_ms_per_step": max(link["both_at_once"]["h2d_ms"], link["both_at_once"]["d2h_ms"]) if link else None},
        "gpu_launches": int(launches),
        "roofline": recs[0] if recs else None,
        "roofline_kernels": recs,
        "effective": {"compulsory_bytes_per_step": compulsory, "compulsory_gbs": compulsory / sec / 1e9,
                      "compulsory_frac_of_measured_hbm": compulsory / sec / 1e9 / peak,
                      "compulsory_frac_of_8TBs": compulsory / sec / 1e9 / NOMINAL_HBM_GBS,
                      "per_access": {"bytes_per_step": per_access, "gbs": per_access / sec / 1e9,
                                     "frac_of_8TBs": per_access / sec / 1e9 / NOMINAL_HBM_GBS,
                                     "frac_of_measured_copy": per_access / sec / 1e9 / peak,
                                     "note": "bytes touched per access (the paper's effective bandwidth); most of them are served on chip, so this is not DRAM traffic"},
                      "distinct_rows_per_s": U / sec},
        "per_step": {"indices": L, "distinct_rows": U, "distinct_hits": U_hit, "index_hit_rate": occ_hit / max(L, 1),
                     "admissions": adm, "evictions": evi, "hot_rows": hot_rows, "hot_row_indices": hot_occ},
        "kernels_ms_per_step": {k: v[0] / K for k, v in ranked},
        "memory_bytes": {"workspace_and_staging": list(h.workspace_bytes())},
    }
    return result


def make_routed(cfg, rank, world, device, sharded_cls=None, backend=None, stream_device=None):
    """The table-wise partition of a model `world` times the configuration's size: every rank owns the configuration's
    tables (its own seed, hence its own rows and index streams), sees the whole batch's bags for them, and the pooled
    vectors / gradients change hands through the ranks' exchange buffers (mpe_forward_routed, mpe_gather_grad).
    Returns (ShardedMpe, Stream of this rank's tables)."""
    from paper_2010_11305_b200 import sharded
    cls = sharded_cls or sharded.ShardedMpe
    rows_global = list(cfg.num_rows) * world
    kw = {} if backend is None else {"backend": backend}
    sm = cls(rows_global, cfg.dim, cfg.bits, cfg.cache_fraction, cfg.ways, cfg.policy, cfg.optimizer, cfg.eps, cfg.init_lo,
             cfg.init_hi, cfg.seed, cfg.batch, device, **kw)
    assert sm.local_rows == list(cfg.num_rows), "equal tables must split evenly over the ranks"
    return sm, wl.Stream(shard_config(cfg, rank), stream_device if stream_device is not None else torch.device("cuda", device))


def routed_step(sm, batch, lr, step):
    """One training step of the partitioned model: forward with the pooled vectors stored into their owners' buffers,
    a rendezvous, the owners' gradients pulled back, backward.  (The gradient buffer keeps what was put there before
    the timed region: the dense model that would write it is outside this library.)"""
    idx, off, _ = batch
    sm.forward(idx, off)
    sm.backward(lr, step)


def run_routed(args, cfg, rank, world, local_rank):
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    sm, stream_gen = make_routed(cfg, rank, world, local_rank)
    total = args.warmup + args.steps
    batches = [stream_gen.batch(s) for s in range(1, total + 1)]
    sm.h.reserve(cfg.batch, max(b[0].numel() for b in batches))
    sm.grad.normal_(0.0, 1e-2)
    torch.distributed.barrier()
    torch.cuda.synchronize(dev)
    for i in range(args.warmup):
        routed_step(sm, batches[i], cfg.lr, i + 1)
    torch.distributed.barrier()
    torch.cuda.synchronize(dev)
    launches0 = sm.h.kernel_launches()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    cs = torch.cuda.current_stream(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.begin()
    e0.record(cs)
    rows = 0
    for i in range(args.warmup, total):
        routed_step(sm, batches[i], cfg.lr, i + 1)
        rows += batches[i][0].numel()
    e1.record(cs)
    torch.distributed.barrier()
    torch.cuda.synchronize(dev)
    sampler.end()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop()
    launches = sm.h.kernel_launches() - launches0
    (ms,), (rows_all,) = aggregate([ms], [float(rows)], world, dev)
    sm.close()
    if rank != 0:
        return None
    K = args.steps
    return {"metric": METRIC, "value": rows_all / (ms * 1e-3), "unit": "rows/s", "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": describe(cfg) + f" on each of {world} ranks ({cfg.num_tables * world} tables in all)",
                       "l2": "inputs larger than L2; a new batch every step",
                       "sharding": "tables partitioned over the ranks; pooled vectors stored into the sample owners' buffers by the pooling "
                                   "kernel, gradients pulled from them (peer loads/stores, two host rendezvous per step)"},
            "clocks": clocks, "gpu_launches": int(launches), "e2e": None, "roofline": None}


def run_tiering(args, local_rank):
    """Effective bandwidth of forward and backward against the cache hit rate, with the low-precision table in HBM
    and in pinned host memory (the experiment of the paper's Section 5.2, on synthetic streams).  One JSON line per point."""
    from dataclasses import replace
    from paper_2010_11305_b200 import binding as mpe
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    base = replace(wl.config(5), bits=args.bits or 16, policy=wl.LRU, cache_fraction=0.01)     # FP16 + 1 % LRU cache
    warm, K = 30, max(args.steps, 5)
    for placement, pname in ((mpe.TABLE_DEVICE, "device"), (mpe.TABLE_HOST, "host")):
        for a in (None, 0.6, 0.8, 0.95, 1.05, 1.2, 1.4):
            cfg = replace(base, zipf=[a] * base.num_tables, name=f"{pname}-{'uniform' if a is None else 'z%g' % a}")
            h = mpe.Mpe(cfg.num_rows, cfg.dim, cfg.bits, cfg.cache_fraction, cfg.ways, cfg.policy, cfg.optimizer, cfg.eps,
                        cfg.init_lo, cfg.init_hi, cfg.seed, local_rank, placement)
            st = wl.Stream(cfg, dev)
            out = torch.empty(cfg.batch, cfg.num_tables * cfg.dim, device=dev)
            cs = torch.cuda.current_stream(dev)
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(3 * K)]
            s0 = None
            for step in range(1, warm + K + 1):
                idx, off, grad = st.batch(step)
                j = step - warm - 1
                if j == 0:
                    torch.cuda.synchronize(dev)
                    s0 = np.sum([h.stats(t) for t in range(cfg.num_tables)], axis=0).astype(np.int64)
                if j >= 0:
                    ev[3 * j].record(cs)
                h.forward(idx, off, cfg.batch, out, cs.cuda_stream)
                if j >= 0:
                    ev[3 * j + 1].record(cs)
                h.backward(grad, cfg.lr, step)
                if j >= 0:
                    ev[3 * j + 2].record(cs)
            torch.cuda.synchronize(dev)
            ds = (np.sum([h.stats(t) for t in range(cfg.num_tables)], axis=0).astype(np.int64) - s0) / K
            L, occ_hit, U, U_hit, adm, evi = (float(ds[i]) for i in range(6))
            fwd_ms = float(np.median([ev[3 * j].elapsed_time(ev[3 * j + 1]) for j in range(K)]))
            bwd_ms = float(np.median([ev[3 * j + 1].elapsed_time(ev[3 * j + 2]) for j in range(K)]))
            d, T, B = cfg.dim, cfg.num_tables, cfg.batch
            rb, fb = d * cfg.bits // 8 + (0 if cfg.bits == 16 else 8), 4 * d
            fwd_bytes = 4 * L + occ_hit * fb + (L - occ_hit) * rb + 4 * B * T * d
            bwd_bytes = L * fb + U_hit * 2 * fb + (U - U_hit) * 2 * rb + 4 * U_hit + evi * (fb + rb) + adm * fb
            print(json.dumps({"placement": pname, "stream": "uniform" if a is None else f"zipf {a}", "index_hit_rate": occ_hit / max(L, 1),
                              "fwd_ms": fwd_ms, "bwd_ms": bwd_ms, "fwd_effective_gbs": fwd_bytes / fwd_ms / 1e6,
                              "bwd_effective_gbs": bwd_bytes / bwd_ms / 1e6, "rows_per_s": L / (fwd_ms + bwd_ms) * 1e3}), flush=True)
            h.close()
            del st


def sample_tables(cfg, budget_rows):
    """How many tables of the configuration the CPU oracle can process in the time budget (~10-30 s)."""
    per_table = cfg.batch * (cfg.bag[1] if cfg.bag[0] != "fixed" else cfg.bag[1])
    n = int(max(1, min(cfg.num_tables, budget_rows // max(per_table, 1))))
    return list(range(n))


def cpu_model():
    try:
        for line in open("/proc/cpuinfo"):
            if line.lower().startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def _oracle_args(cfg):
    return (cfg.num_rows, cfg.dim, cfg.bits, cfg.cache_fraction, cfg.ways, cfg.policy, cfg.optimizer, cfg.eps, cfg.init_lo,
            cfg.init_hi, cfg.seed)


def run_oracle(cfg, steps, warmup, stream_device, budget_rows=3_000_000):
    """The CPU oracle, as it stands, on ONE host core: `steps` steps over a sample of the tables after `warmup` untimed
    ones (the first step materialises every row it touches, which is not the method's work)."""
    from oracle import mpe_oracle as orc
    tables = sample_tables(cfg, budget_rows // max(steps + warmup, 1))
    o = orc.Oracle(*_oracle_args(cfg))
    mask = np.zeros(cfg.num_tables, np.uint8)
    mask[tables] = 1
    o.set_table_mask(mask)
    st = wl.Stream(cfg, stream_device)
    rows, secs = 0, 0.0
    for s in range(1, warmup + steps + 1):
        idx, off, grad = (x.cpu().numpy() for x in st.batch(s))
        t0 = time.perf_counter()
        o.forward(idx, off, cfg.batch)
        o.backward(grad, cfg.lr, s)
        dt = time.perf_counter() - t0
        if s > warmup:
            secs += dt
            rows += int(sum(off[(t + 1) * cfg.batch] - off[t * cfg.batch] for t in tables))
    return {"value": rows / secs if secs > 0 else None, "unit": "rows/s", "cores": 1, "kind": "oracle",
            "sample": f"{len(tables)} of {cfg.num_tables} tables, {steps} step(s) after {warmup} warm-up, "
                      f"{rows} index rows in {secs:.1f} s",
            "seconds": secs, "rows": rows, "cpu": cpu_model(), "nproc": os.cpu_count()}


def _oracle_worker(rank, root, oargs, tables, files, batch, lr, warmup, gate, q):
    """One process of the all-cores leg: the unchanged oracle on its own tables (tables are independent units)."""
    sys.path.insert(0, root)
    from oracle import mpe_oracle as orc
    o = orc.Oracle(*oargs)
    mask = np.zeros(len(oargs[0]), np.uint8)
    mask[tables] = 1
    o.set_table_mask(mask)
    data = [tuple(np.load(f, mmap_mode="r") for f in fs) for fs in files]
    rows, t0 = 0, None
    for s, (idx, off, grad) in enumerate(data, start=1):
        if s == warmup + 1:
            gate.wait()                              # every process starts its timed steps together
            t0 = time.time()
        o.forward(idx, off, batch)
        o.backward(grad, lr, s)
        if s > warmup:
            rows += int(sum(off[(t + 1) * batch] - off[t * batch] for t in tables))
    q.put((rank, rows, t0, time.time()))


def run_oracle_all_cores(cfg, steps, warmup, stream_device, tables_per_core=1):
    """The same oracle over all host cores: one process per core, each with its own tables; rows of all / wall time."""
    import multiprocessing as mp
    import shutil
    import tempfile
    ncores = os.cpu_count() or 1
    workers = max(1, min(ncores, cfg.num_tables))
    per = max(1, min(tables_per_core, cfg.num_tables // workers))
    assign = [list(range(w * per, (w + 1) * per)) for w in range(workers)]
    base = "/dev/shm" if os.path.isdir("/dev/shm") else None
    tmp = tempfile.mkdtemp(prefix="mpe_oracle_", dir=base)
    try:
        st = wl.Stream(cfg, stream_device)
        files = []
        for s in range(1, warmup + steps + 1):
            fs = []
            for name, x in zip(("idx", "off", "grad"), st.batch(s)):
                f = os.path.join(tmp, f"{name}{s}.npy")
                np.save(f, x.cpu().numpy())
                fs.append(f)
            files.append(fs)
        del st
        ctx = mp.get_context("spawn")
        gate, q = ctx.Barrier(workers), ctx.Queue()
        procs = [ctx.Process(target=_oracle_worker, args=(w, ROOT, _oracle_args(cfg), assign[w], files, cfg.batch, cfg.lr, warmup, gate, q))
                 for w in range(workers)]
        for p in procs:
            p.start()
        res, t_give_up = [], time.time() + 600
        while len(res) < len(procs):
            try:
                res.append(q.get(timeout=2))
            except Exception:
                if any(p.exitcode not in (None, 0) for p in procs) or time.time() > t_give_up:
                    for p in procs:
                        p.terminate()
                    raise RuntimeError("an oracle process ended early")
        for p in procs:
            p.join(timeout=60)
    finally:
        shutil.rmtree(tmp, ignore_errors=True)
    rows = sum(r[1] for r in res)
    wall = max(r[3] for r in res) - min(r[2] for r in res)
    return {"value": rows / wall if wall > 0 else None, "unit": "rows/s", "cores": workers, "kind": "oracle, one process per core over disjoint tables",
            "sample": f"{workers * per} of {cfg.num_tables} tables ({per} per process), {steps} step(s) after {warmup} warm-up, "
                      f"{rows} index rows in {wall:.1f} s of wall time",
            "seconds": wall, "rows": rows, "cpu": cpu_model(), "nproc": ncores}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=6)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--routed", action="store_true", help="with --gpus N > 1: partition the tables over the ranks and time the step with the "
                    "exchange of pooled vectors and gradients inside it (default: every rank trains its own tables, no exchange)")
    ap.add_argument("--no-prepare", action="store_true", help="do not sort the next batch ahead of time (mpe_prepare)")
    ap.add_argument("--sweep5", action="store_true", help="run every point of the policy/skew sweep (configuration 5): one JSON line per point")
    ap.add_argument("--tiering", action="store_true", help="forward/backward effective bandwidth vs hit rate, table in HBM and in host memory")
    ap.add_argument("--sweep-assoc", action="store_true", help="associativity sweep (1..32 ways, LRU and LFU) on configuration 5's shape")
    ap.add_argument("--bits", type=int, default=None, help="override the table precision: 16 (FP16), 8, 4 or 2")
    ap.add_argument("--policy", default=None, choices=["lru", "lfu"], help="override the replacement policy")
    ap.add_argument("--tables", type=int, default=None, help="profiling aid: keep only the first TABLES tables")
    ap.add_argument("--rows-div", type=int, default=1, help="profiling aid: divide every table's row count")
    ap.add_argument("--batch-div", type=int, default=1, help="profiling aid: divide the batch size")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    def make_cfg():
        c = wl.config(args.config)
        if args.tables is not None or args.rows_div != 1 or args.batch_div != 1:
            c = wl.scaled(c, rows_div=args.rows_div, batch_div=args.batch_div, tables=args.tables)
        if args.bits is not None:
            c.bits = args.bits
            c.name += f"/bits{args.bits}"
        if args.policy is not None:
            c.policy = wl.LRU if args.policy == "lru" else wl.LFU
            c.name += f"/{args.policy}"
        return c

    cfg = make_cfg()

    if args.impl == "reference":
        if rank != 0:
            return
        dev = "cuda" if torch.cuda.is_available() else "cpu"
        r = run_oracle(cfg, args.steps, min(args.warmup, 1), dev, budget_rows=2_000_000)
        line = {"metric": METRIC, "impl": "reference", "value": r["value"], "unit": "rows/s", "n_gpus": args.gpus,
                "steps": args.steps, "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * r["seconds"] / max(args.steps, 1),
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": describe(cfg)},
                "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample", "cpu", "nproc")},
                "e2e": {"value": r["value"], "unit": "rows/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    if args.tiering:
        run_tiering(args, local_rank)
        return
    if args.sweep_assoc:
        # hit rate per (ways, policy, cache size) on a Zipf(1.05) stream: the layout of the paper's hit-rate table
        from dataclasses import replace
        args.e2e_steps = 0
        args.warmup = max(args.warmup, 50)
        for frac in (0.05, 0.10, 0.30, 0.50):
            for policy in (wl.LRU, wl.LFU):
                for ways in (1, 2, 4, 8, 16, 32):
                    point = replace(wl.config(5), name=f"c{frac:g}-{'lru' if policy == wl.LRU else 'lfu'}-{ways}way", ways=ways,
                                    policy=policy, cache_fraction=frac)
                    r = run_ours(args, point, 0, 1, local_rank)
                    print(json.dumps({"point": point.name, "cache_fraction": frac, "policy": "lru" if policy == wl.LRU else "lfu",
                                      "ways": ways, "index_hit_rate": r["per_step"]["index_hit_rate"], "ms_per_step": r["ms_per_step"],
                                      "rows_per_s": r["value"]}), flush=True)
        return
    if args.sweep5:
        # hit rate, rows/s and effective GB/s per point; 50 warm-up steps fill the caches, then `--steps` are timed
        args.e2e_steps = 0
        args.warmup = max(args.warmup, 50)
        for point in wl.sweep5():
            r = run_ours(args, point, 0, 1, local_rank)
            print(json.dumps({"point": point.name, "rows_per_s": r["value"], "ms_per_step": r["ms_per_step"],
                              "index_hit_rate": r["per_step"]["index_hit_rate"], "effective_gbs": r["effective"]["per_access"]["gbs"],
                              "compulsory_gbs": r["effective"]["compulsory_gbs"],
                              "distinct_rows": r["per_step"]["distinct_rows"], "gpu_launches": r["gpu_launches"]}), flush=True)
        return
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    result = run_routed(args, cfg, rank, world, local_rank) if (args.routed and world > 1) else run_ours(args, cfg, rank, world, local_rank)
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline and result is not None:
            sdev = torch.device("cuda", local_rank)
            r = run_oracle(make_cfg(), 3, 1, sdev, budget_rows=10_000_000)
            result["cpu_baseline"] = {k: r[k] for k in ("value", "unit", "cores", "kind", "sample", "cpu", "nproc")}
            try:
                r = run_oracle_all_cores(make_cfg(), 3, 1, sdev)
                result["cpu_baseline"]["all_cores"] = {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")}
            except Exception as exc:       # a box that cannot spawn processes still reports the one-core figure
                result["cpu_baseline"]["all_cores"] = {"unavailable": repr(exc)}
        print(json.dumps(result))
    if world > 1:
        torch.distributed.barrier()
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
