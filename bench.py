"""Benchmark of the ByzShield aggregation path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-extra] [--no-sweep]

One step = one fused vote + coordinate-wise median (bz_vote_median) over a resident batch of
replicated file gradients: K = 15 workers, r = 3, l = 5, f = 25 files, d = 11.2 M coordinates,
q = 3 Byzantine workers at the worst-case placement sending -100 x the true gradient.
With N > 1 every rank aggregates its own coordinate slab of the same size (the path needs no collective);
the Multi-Krum leg adds its one all-reduce of the 49 x 49 distance matrix.  `--gpus N` without a launcher
starts the N ranks itself.  Rank 0 prints ONE JSON line.  `--impl reference` times the CPU checker instead.
`--coords`, `--no-e2e`, `--no-cpu`, `--op` shrink the run for profiler captures; their JSON line names the
smaller workload and is not a benchmark value.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "aggregated gradient coordinates/sec (fused vote+median)"
UNIT = "coordinates/s"
WORKLOAD = dict(l=5, r=3, q=3, d=11_200_000, attack="reversed", seed=0)
MULTIKRUM = dict(l=7, r=3, q=5, d=11_200_000, attack="alie", seed=0, c=5, m=44)
BULYAN = dict(l=5, r=5, q=6, d=25_000_000, attack="constant", seed=0, c=4, heavy=0.01)

# DRAM bytes per launch of the dominant kernel from an ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum, scaled to a full launch), or None when no capture of the current kernel exists.
TRAFFIC_BYTES_PER_LAUNCH = 3_422_552_000  # (600.02 + 11.15) MB at d = 2 M, scaled by 5.6 to d = 11.2 M


def workload_name(cfg):
    return ("K=%d r=%d l=%d f=%d d=%s fp32, q=%d Byzantine (worst-case placement) sending -100 x gradient; "
            "fused vote + coordinate-wise median" % (cfg["r"] * cfg["l"], cfg["r"], cfg["l"], cfg["l"] ** 2,
                                                     ("%.1fM" % (cfg["d"] / 1e6)), cfg["q"]))


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy read+write)"
    except Exception:
        return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML (read-only) from start() to stop().
    mark()/unmark() bracket a region of interest inside the run; both summaries are reported."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, torch_index: int):
        self.samples, self.max_mhz = [], None      # (monotonic time, MHz, reason bits)
        self.marks = []
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = str(torch.cuda.get_device_properties(torch_index).uuid)
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid) if not uuid.startswith("GPU-") else uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(torch_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # NVML missing: report that no clocks were seen
            self.nv = None
            log("clock sampling unavailable:", e)

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                self.samples.append((time.monotonic(), mhz, bits))
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def mark(self):
        self.marks.append([time.monotonic(), None])

    def unmark(self):
        self.marks[-1][1] = time.monotonic()

    def _summary(self, rows):
        reasons = set()
        for _, _, bits in rows:
            for bit, name in self.REASONS.items():
                if bits & bit:
                    reasons.add(name)
        return {"sm_mhz": (statistics.median([m for _, m, _ in rows]) if rows else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(reasons), "samples": len(rows)}

    def window(self, t0, t1):
        """Clocks between two time.monotonic() stamps."""
        return self._summary([r for r in self.samples if t0 <= r[0] <= t1])

    def summary(self):
        """Clocks over the marked regions (warm-up + timed steps of the headline), and over the whole run."""
        inside = [s for s in self.samples if any(a <= s[0] <= (b if b is not None else s[0]) for a, b in self.marks)]
        out = self._summary(inside)
        out["region"] = "warm-up and timed steps of the headline kernel"
        whole = self._summary(self.samples)
        # under load = samples at or above 90 % of the maximum clock or with a reason active
        out["whole_run"] = whole
        return out


def make_inputs(bz, inputs, cfg, device, seed_offset=0):
    """Assignment and Byzantine set through the library, synthetic replicas on the device."""
    l, r, q, d = cfg["l"], cfg["r"], cfg["q"], cfg["d"]
    _, fw, mask = bz.assign_mols(l, r)
    cmax, byz, _ = bz.worst_case(mask, l * l, r, q)
    g = inputs.true_gradients(l * l, d, seed=cfg["seed"] + seed_offset, heavy_tail_frac=cfg.get("heavy", 0.0), device=device)
    rep = inputs.build_replicas(g, fw, byz, cfg["attack"])
    del g
    return rep, fw, byz, cmax


def timed_calls(torch, fn, steps, warmup):
    """Device time of each of `steps` calls (CUDA events on the current stream): ms as best / median / mean."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    ev[0].record()
    for i in range(steps):
        fn()
        ev[i + 1].record()
    torch.cuda.synchronize()
    each = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
    return {"best": min(each), "median": statistics.median(each), "mean": ev[0].elapsed_time(ev[steps]) / steps}


def timed(torch, fn, steps, warmup):
    return timed_calls(torch, fn, steps, warmup)["mean"]


def e2e_leg(bz, torch, dist, world, rep, out, device, steps):
    """The same aggregation through the host entry point: pinned host buffers, copies inside the timing."""
    r, f, d = rep.shape
    rep_host = torch.empty((r, f, d), dtype=torch.float32, pin_memory=True)
    rep_host.copy_(rep)
    out_host = torch.empty(d, dtype=torch.float32, pin_memory=True)
    ws = torch.empty((r * f + 1) * ((d + 63) // 64 * 64) * 4 + 256, dtype=torch.uint8, device=device)
    step = lambda: bz.vote_median_host(rep_host, out_host, ws)
    step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    n = max(2, min(5, steps))
    t0 = time.perf_counter()
    for _ in range(n):
        step()
    torch.cuda.synchronize()
    secs = torch.tensor([(time.perf_counter() - t0) / n], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(secs, op=dist.ReduceOp.MAX)
    matches = bool(torch.equal(out_host.to(device), out))
    return {"value": world * d / float(secs.item()), "unit": UNIT, "h2d_bytes_per_step": r * f * d * 4,
            "d2h_bytes_per_step": d * 4, "steps": n, "matches_device_result": matches}, rep_host


def multikrum_leg(bz, inputs, torch, dist, world, rank, device, steps, warmup, peak, sampler=None):
    """Multi-Krum from the replicas (vote + distances in one pass, selection, mean) at K = 21, (l, r) = (7, 3),
    f = 49, d = 11.2 M per GPU, q = 5 with the ALIE payload, (c, m) = (5, 44).  With several ranks every rank owns
    a slab of that size and the partial distance matrices are added by one all-reduce."""
    from paper_2010_04902_b200 import sharding
    cfg = dict(MULTIKRUM)
    rep, fw, byz, cmax = make_inputs(bz, inputs, cfg, device, seed_offset=rank)
    l, r, d, c, m = cfg["l"], cfg["r"], cfg["d"], cfg["c"], cfg["m"]
    f = l * l
    voted = torch.empty((f, d), dtype=torch.float32, device=device)
    out = torch.empty(d, dtype=torch.float32, device=device)
    ws = bz.alloc_workspace(bz.OP_MULTIKRUM, 0, f, d, c, m, device=device)
    dmat = torch.empty((f, f), dtype=torch.float64, device=device)
    if world == 1:
        step = lambda: bz.vote_multikrum(rep, c, m, voted=voted, workspace=ws, out=out, dist=dmat)
    else:
        step = lambda: sharding.vote_multikrum(rep, c, m)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
        torch.cuda.synchronize()
    n0 = bz.kernel_launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    t_begin = time.monotonic()
    ev[0].record()
    for i in range(steps):
        res = step()
        ev[i + 1].record()
    torch.cuda.synchronize()
    t_end = time.monotonic()
    launches = bz.kernel_launch_count() - n0
    ms_total = torch.tensor([ev[0].elapsed_time(ev[steps])], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(ms_total, op=dist.ReduceOp.MAX)
    ms = float(ms_total.item()) / steps
    each = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
    alg_bytes = (4 * r * f + 4 * f + 4 * m + 4) * d
    gbs = alg_bytes / (ms * 1e-3) / 1e9
    rec = {"metric": "aggregated gradient coordinates/sec (vote + Multi-Krum from the replicas)", "value": world * d / (ms * 1e-3),
           "unit": UNIT, "ms_per_step": ms, "ms_best": min(each), "ms_median": statistics.median(each), "steps": steps,
           "workload": "K=21 r=3 l=7 f=49 d=11.2M per GPU, q=5 ALIE, c=5 m=44; bz_vote_multikrum"
                       + ("" if world == 1 else " per coordinate slab + one all-reduce of the 49x49 fp64 matrix (%s)"
                          % os.environ.get("BZ_BENCH_DIST_BACKEND", "nccl")),
           "c_max": cmax, "gpu_launches": int(launches),
           "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                        "algorithmic_bytes_per_step": alg_bytes,
                        "kernels": "pairdist_i8_kernel<49,25,3,25,3,1> (vote + integer MMA distances), mean_rows_kernel"},
           "status_bits (0 = the integer kernel's distances stood)": bz.pairdist_status(ws, f) if world == 1 else None}
    # this pipeline (tensor cores, conversion and HBM all busy) reaches the board's power limit within tenths of a
    # second: the later steps run at lower SM clocks than the first ones, and both are reported
    quarter = max(1, steps // 4)
    rec["ms_first_quarter"] = sum(each[:quarter]) / quarter
    rec["ms_last_quarter"] = sum(each[-quarter:]) / quarter
    if sampler is not None:
        rec["clocks"] = sampler.window(t_begin, t_end)
    if world == 1:
        return rec, (rep, voted, out, dmat, res[1])
    del rep
    return rec, None


def krum_parity(bz, torch, np, oracle, rep, voted, out, dmat, sel, cfg):
    """The timed Multi-Krum result against the CPU checker on ALL rows and coordinates."""
    r, f, d = rep.shape
    t0 = time.perf_counter()
    want_voted = np.empty((f, d), np.float32)
    for i0 in range(0, f, 7):
        want_voted[i0:i0 + 7] = oracle.vote(rep[:, i0:i0 + 7].cpu().numpy())
    voted_ok = bool(np.array_equal(voted.cpu().numpy().view(np.uint32), want_voted.view(np.uint32)))
    want_out, want_sel, want_D = oracle.multikrum(want_voted, cfg["c"], cfg["m"])
    got_D = dmat.cpu().numpy()
    nz = want_D > 0
    err = float((np.abs(got_D[nz] - want_D[nz]) / want_D[nz]).max())
    zeros_ok = bool((got_D[~nz] == 0).all())
    scores = np.sort(oracle.krum_scores(want_D, cfg["c"]), kind="stable")
    m = cfg["m"]
    gap = float((scores[m] - scores[m - 1]) / scores[m])
    got_out = out.cpu().numpy().astype(np.float64)
    rel_l2 = float(np.linalg.norm(got_out - want_out) / np.linalg.norm(want_out))
    rec = {"voted_bit_exact": voted_ok, "selected_equal": sel.cpu().tolist() == want_sel.tolist(),
           "gpu_max_rel_error_in_D": err, "identical_rows_exactly_zero": zeros_ok,
           "oracle_min_rel_score_gap_at_selection_boundary": gap, "out_rel_l2": rel_l2,
           "out_bit_exact": bool(np.array_equal(out.cpu().numpy(), want_out)),
           "rows": f, "coordinates": d, "oracle_seconds": time.perf_counter() - t0}
    if not (voted_ok and rec["selected_equal"] and err <= 1e-7 and zeros_ok and rel_l2 <= 1e-5):
        raise RuntimeError("Multi-Krum bench output differs from the CPU checker: %r" % (rec,))
    return rec


def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    from paper_2010_04902_b200 import binding as bz
    from paper_2010_04902_b200 import build as bz_build
    from paper_2010_04902_b200 import inputs

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the aggregation path has no CPU fallback")
    # one rank per GPU.  (BZ_BENCH_DIST_BACKEND=gloo lets several ranks share the GPUs there are - a functional check of
    # the multi-rank path on a smaller box, not a measurement: NCCL wants a device per rank.)
    backend = os.environ.get("BZ_BENCH_DIST_BACKEND", "nccl")
    local_rank = local_rank if backend == "nccl" else local_rank % torch.cuda.device_count()
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("NCCL_DEBUG", "INFO")   # NCCL's own account of the transport (NVLS, rings) goes to stderr
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=device)
        else:
            dist.init_process_group(backend)
    if rank == 0:
        bz_build.build()
    if world > 1:
        dist.barrier()
    bz.lib()
    peak, peak_src = measured_peaks()
    sampler = ClockSampler(local_rank).start()

    cfg = dict(WORKLOAD)
    if args.coords > 0:
        cfg["d"] = args.coords
    l, r, d = cfg["l"], cfg["r"], cfg["d"]
    f = l * l
    rep, fw, byz, cmax = make_inputs(bz, inputs, cfg, device, seed_offset=rank)
    out = torch.empty(d, dtype=torch.float32, device=device)
    step = lambda: bz.vote_median(rep, out)

    # ---- timed region: exactly K steps between barriers, device time, max over ranks ----------------
    sampler.mark()
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
        torch.cuda.synchronize()
    n0 = bz.kernel_launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    ev[0].record()
    for i in range(args.steps):
        step()
        ev[i + 1].record()
    torch.cuda.synchronize()
    sampler.unmark()
    launches = bz.kernel_launch_count() - n0
    staged = bz.last_path() == bz.PATH_STAGED
    if world > 1:
        dist.barrier()
    ms_total = torch.tensor([ev[0].elapsed_time(ev[args.steps])], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(ms_total, op=dist.ReduceOp.MAX)
    ms_step = float(ms_total.item()) / args.steps
    each = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    value = world * d / (ms_step * 1e-3)

    e2e, rep_host = (None, None)
    if not args.no_e2e:
        e2e, rep_host = e2e_leg(bz, torch, dist, world, rep, out, device, args.steps)

    result = None
    if rank == 0:
        alg_bytes = (4 * r * f + 4) * d
        achieved = alg_bytes / (ms_step * 1e-3) / 1e9
        traffic = TRAFFIC_BYTES_PER_LAUNCH if args.coords == 0 else None
        result = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "ms_best": min(each), "ms_median": statistics.median(each),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32",
            "data": "synthetic",
            "config": {"workload": workload_name(cfg), "coordinates_per_gpu": d, "c_max": cmax,
                       "byzantine_workers": [int(u) for u in byz],
                       "l2": "inputs are %.2f GB per step, far larger than the 126 MB L2; no flush needed" % (4 * r * f * d / 1e9),
                       "parallelism": ("coordinate slabs, no collective" + ("" if backend == "nccl" else " (%s backend, ranks sharing GPUs: "
                                       "functional check only)" % backend)) if world > 1 else "single GPU"},
            "e2e": e2e,
            "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": traffic, "peak_source": peak_src, "frac_of_nominal_8TBs": achieved / 8000.0,
                         "algorithmic_bytes_per_launch": alg_bytes,
                         "kernel": ("vote_median_tma_kernel<3,25,25,3>" if staged else "vote_median_kernel (register path)")
                                   + " (one launch per step)"},
        }

    # ---- CPU baseline and parity of the timed output (single-GPU run only) ----------------------------
    if rank == 0 and world == 1 and not args.no_cpu:
        import oracle
        cores = oracle.num_threads()
        probe = rep[:, :, :min(d, 200_000)].cpu().numpy()
        t0 = time.perf_counter()
        oracle.vote_median(probe)
        rate = probe.shape[2] / (time.perf_counter() - t0)
        n_sample = int(min(d, max(200_000, rate * 15.0)))
        sample = (rep_host[:, :, :n_sample] if rep_host is not None else rep[:, :, :n_sample].cpu()).contiguous().numpy()
        t0 = time.perf_counter()
        want = oracle.vote_median(sample)
        dt = time.perf_counter() - t0
        got = out[:n_sample].cpu().numpy()
        parity = bool(np.array_equal(got.view(np.uint32), want.view(np.uint32)))
        result["cpu_baseline"] = {"value": n_sample / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
                                  "sample": "first %d of %d coordinates of the same replicas (all %d rows)" % (n_sample, d, r * f)}
        result["parity"] = {"bit_exact_vs_oracle_on_sample": parity, "sample_coordinates": n_sample}
        if not parity:
            raise RuntimeError("bench output differs from the CPU checker")
    if rank == 0 and world == 1 and not args.no_extra:
        result["streaming_probe"] = probe_leg(bz, torch, rep, peak)
    del rep_host, rep, out
    torch.cuda.empty_cache()

    # ---- the metric's second aggregator: Multi-Krum (every rank; one all-reduce when N > 1) --------------
    if not args.no_extra and args.coords == 0:
        sec, keep = multikrum_leg(bz, inputs, torch, dist, world, rank, device, max(5, min(args.steps, 50)), 10, peak, sampler)
        if rank == 0:
            result["secondary"] = sec
            if world == 1 and not args.no_cpu:
                import oracle
                result["secondary"]["parity"] = krum_parity(bz, torch, np, oracle, *keep, MULTIKRUM)
        del keep
        torch.cuda.empty_cache()

    # ---- N > 1: the exhaustive worst-case search dealt to the ranks (one gather of the shares' maxima) -------
    if world > 1 and not args.no_extra and args.coords == 0:
        from paper_2010_04902_b200 import sharding
        _, _, mask75 = bz.assign_mols(7, 5)
        sharding.worst_case(mask75, 49, 5, 9)                      # warm-up (and the binomial table)
        dist.barrier()
        t0 = time.perf_counter()
        c13, set13, n13 = sharding.worst_case(mask75, 49, 5, 13)
        dist.barrier()
        dt = time.perf_counter() - t0
        if rank == 0:
            result["worst_case_sharded"] = {"K": 35, "f": 49, "r": 5, "q": 13, "subsets": n13, "c_max": c13, "argmax": set13,
                                            "seconds_wall_all_ranks": dt, "subsets_per_s": n13 / dt,
                                            "sharding": "subsets dealt to the ranks in fixed-size runs; one all_gather of (c_max, argmax)"}

    if rank == 0 and world == 1 and not args.no_extra and args.coords == 0:
        result["config1"] = config1_leg(bz, inputs, torch, device)
        result["unaligned_d"] = unaligned_leg(bz, inputs, torch, device, peak)
        result["other_paths"] = extra_paths(bz, inputs, torch, device)
        if not args.no_sweep:
            result["sweep"] = sweep(bz, inputs, torch, device, peak)

    sampler.stop()
    if rank == 0:
        result["clocks"] = sampler.summary()
        result["pipeline_timeouts"] = bz.pipeline_timeouts()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(result), flush=True)


def probe_leg(bz, torch, rep, peak):
    """Read-only streaming bandwidth of this GPU, measured with the library's own probe kernels on the headline's
    replicas (3.36 GB, far larger than L2): the second denominator beside the copy peak.  Two ways of reading:
    128-bit loads into registers, and the bulk-copy engine filling a ring in shared memory (how the staged kernels read)."""
    sink = torch.zeros(1, dtype=torch.int64, device=rep.device)
    nbytes = rep.numel() * 4
    out = {"bytes": nbytes, "copy_peak_GBs": peak}
    for name, staged in (("register_loads", False), ("bulk_copy_ring", True)):
        t = timed_calls(torch, lambda: bz.stream_probe(rep, sink, staged=staged), 20, 3)
        out[name] = {"ms_best": t["best"], "ms_median": t["median"], "read_GBs_best": nbytes / (t["best"] * 1e-3) / 1e9,
                     "read_GBs_median": nbytes / (t["median"] * 1e-3) / 1e9}
    out["read_GBs_best"] = max(out["register_loads"]["read_GBs_best"], out["bulk_copy_ring"]["read_GBs_best"])
    return out


def config1_leg(bz, inputs, torch, device):
    """K = 15, (l, r) = (5, 3), d = 100 000, q = 2 with the ALIE payload: vote then median, and the fused pass.
    30 MB of replicas fit the 126 MB L2, so the case is reported warm (same buffers every call) and cold (rotating
    over 8 copies, 240 MB); at this size a call is bound by launch latency either way, so the calls are also
    replayed from a CUDA graph, which takes the host out of the measurement."""
    cfg = dict(l=5, r=3, q=2, d=100_000, attack="alie", seed=0)
    rep0, fw, byz, cmax = make_inputs(bz, inputs, cfg, device)
    f, d = 25, cfg["d"]
    reps = [rep0] + [rep0.clone() for _ in range(7)]
    voted = torch.empty((f, d), dtype=torch.float32, device=device)
    out = torch.empty(d, dtype=torch.float32, device=device)
    res = {"workload": "K=15 r=3 l=5 f=25 d=100000, q=2 ALIE (c_max=%d)" % cmax, "bytes_per_call": 4 * 3 * f * d}

    def both(i):
        bz.vote(reps[i], voted)
        bz.median(voted, out)

    def fused(i):
        bz.vote_median(reps[i], out)

    for name, fn in (("vote_then_median", both), ("fused", fused)):
        rec = {}
        for mode, idx in (("warm", [0] * 8), ("cold", list(range(8)))):
            state = {"k": 0}

            def call():
                fn(idx[state["k"] % 8])
                state["k"] += 1
            t = timed_calls(torch, call, 64, 8)
            rec[mode + "_us_median"] = t["median"] * 1e3
            rec[mode + "_us_best"] = t["best"] * 1e3
            # the same 8 calls as one CUDA graph, replayed
            try:
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    for i in idx:
                        fn(i)
                    side.synchronize()
                    graph = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(graph, stream=side):
                        for i in idx:
                            fn(i)
                torch.cuda.synchronize()
                t = timed_calls(torch, graph.replay, 20, 3)
                rec[mode + "_graph_us_per_call_median"] = t["median"] * 1e3 / 8
                del graph
            except Exception as e:  # capture refused: the plain loop's numbers stand alone
                rec[mode + "_graph"] = "not captured: %s" % (str(e).splitlines()[0][:120],)
                torch.cuda.synchronize()
        rec["coordinates_per_s_cold"] = d / (rec["cold_us_median"] * 1e-6)
        res[name] = rec
    return res


def unaligned_leg(bz, inputs, torch, device, peak):
    """The headline shape at a length that is not a multiple of 4 (d = 11 173 962): rows then start off 16-byte
    boundaries, so the staged and 128-bit kernels do not apply and the scalar register kernels answer."""
    d = 11_173_962
    cfg = dict(WORKLOAD, d=d)
    rep, fw, byz, cmax = make_inputs(bz, inputs, cfg, device)
    out = torch.empty(d, dtype=torch.float32, device=device)
    voted = torch.empty((25, d), dtype=torch.float32, device=device)
    t = timed_calls(torch, lambda: bz.vote_median(rep, out), 10, 3)
    path = bz.last_path()
    tv = timed_calls(torch, lambda: bz.vote(rep, voted), 10, 3)
    nb = (4 * 3 * 25 + 4) * d
    names = {bz.PATH_STAGED: "staged", bz.PATH_REGISTERS: "registers", bz.PATH_GENERIC: "generic", bz.PATH_TENSOR: "tensor",
             bz.PATH_FP32: "fp32", bz.PATH_FP64: "fp64"}
    rec = {"d": d, "path": names.get(path, path),
           "vote_median_ms_best": t["best"], "vote_median_ms_median": t["median"],
           "vote_median_frac_of_measured_hbm": nb / (t["median"] * 1e-3) / 1e9 / peak,
           "vote_ms_median": tv["median"], "vote_frac_of_measured_hbm": (4 * 3 * 25 + 4 * 25) * d / (tv["median"] * 1e-3) / 1e9 / peak}
    # the other kernels on the same rows (f = 25, c = 3): median, distances, Multi-Krum, Bulyan, and both from the replicas
    f, c = 25, 3
    ws = bz.alloc_workspace(bz.OP_MULTIKRUM, 0, f, d, c, f - c, device=device)
    tm = timed_calls(torch, lambda: bz.median(voted, out), 10, 3)
    rec["median_ms_median"] = tm["median"]
    rec["median_frac_of_measured_hbm"] = (4 * f + 4) * d / (tm["median"] * 1e-3) / 1e9 / peak
    tp = timed_calls(torch, lambda: bz.pairdist(voted, ws), 5, 2)
    rec["pairdist_ms_median"] = tp["median"]
    rec["pairdist_path"] = names.get(bz.last_path(), bz.last_path())
    rec["multikrum_ms_median"] = timed_calls(torch, lambda: bz.multikrum(voted, c, f - c, workspace=ws, out=out), 5, 2)["median"]
    rec["bulyan_ms_median"] = timed_calls(torch, lambda: bz.bulyan(voted, c, workspace=ws, out=out), 5, 2)["median"]
    rec["vote_multikrum_ms_median"] = timed_calls(torch, lambda: bz.vote_multikrum(rep, c, f - c, voted=voted, workspace=ws, out=out), 5, 2)["median"]
    rec["vote_bulyan_ms_median"] = timed_calls(torch, lambda: bz.vote_bulyan(rep, c, voted=voted, workspace=ws, out=out), 5, 2)["median"]
    rec["note"] = ("rows of 11 173 962 floats start on 8-byte boundaries: no 16-byte aligned leading dimension, so the staged (TMA) "
                   "kernels and the integer distance kernel do not apply; a caller that pads each row to a multiple of 4 floats gets them")
    return rec


SWEEP_SHAPES = [(5, 3, 3), (5, 5, 6), (7, 3, 5), (7, 5, 5), (7, 7, 6)]   # (l, r, q of the timed inputs)


def sweep(bz, inputs, torch, device, peak):
    """Feasible (l, r) x d in {1 M, 10 M, 100 M}: fused vote + median and Multi-Krum from the replicas (c = c_max of the
    timed q, m = f - c), ms as best / median of 10 calls, coordinates/s and fraction of the measured copy peak; and for
    every assignment the exhaustive worst-case count for q = 1 .. floor((K-1)/2) (all subsets while C(K, q) <= 2^36,
    one set per translation orbit beyond)."""
    cells, counts = [], []
    cells.append({"l": 5, "r": 7, "status": "infeasible: r > l (at most l - 1 Latin squares, l parallel classes; Sec. 4.1.1, Eq. 7)"})
    c_of = {}
    for l, r, q in SWEEP_SHAPES:
        K, f = l * r, l * l
        _, fw, mask = bz.assign_mols(l, r)
        ws_wc = bz.alloc_workspace(bz.OP_WORST_CASE, r, f)
        ws_orb = bz.alloc_workspace(bz.OP_WORST_CASE_MOLS, r, f)
        cm, methods, n_sets = [], [], 0
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for qq in range(1, (K - 1) // 2 + 1):
            try:
                c_, _, n_ = bz.worst_case(mask, f, r, qq, max_subsets=1 << 36, workspace=ws_wc)
                methods.append("all")
            except bz.BzError as e:
                if e.status != bz.ERR_BUDGET:
                    raise
                c_, _, n_ = bz.worst_case_mols(l, r, qq, workspace=ws_orb)
                methods.append("orbits")
            cm.append(int(c_))
            n_sets += int(n_)
        counts.append({"l": l, "r": r, "K": K, "q": [1, (K - 1) // 2], "c_max": cm, "seconds": time.perf_counter() - t0,
                       "sets_evaluated": n_sets, "first_q_by_orbits": (methods.index("orbits") + 1) if "orbits" in methods else None})
        c_of[(l, r)] = cm[q - 1]
    # the short cells first: the long ones leave the board at its power cap for a while
    for d in (1_000_000, 10_000_000, 100_000_000):
        for l, r, q in SWEEP_SHAPES:
            f = l * l
            cmax_q = c_of[(l, r)]
            need = 4 * d * (r * f + f + 3) * 1.03 + (1 << 28)
            free = torch.cuda.mem_get_info()[0]
            cell = {"l": l, "r": r, "f": f, "d": d, "q": q, "c": cmax_q, "m": f - cmax_q}
            if need > free:
                cell["status"] = "skipped: needs %.0f GB, %.0f GB free" % (need / 1e9, free / 1e9)
                cells.append(cell)
                continue
            cfg = dict(l=l, r=r, q=q, d=d, attack="reversed", seed=d % 1000)
            rep, _, _, _ = make_inputs(bz, inputs, cfg, device)
            out = torch.empty(d, dtype=torch.float32, device=device)
            n_calls = 50 if d <= 1_000_000 else (10 if d <= 10_000_000 else 5)   # short calls: enough of them to outlast clock ramps
            t = timed_calls(torch, lambda: bz.vote_median(rep, out), n_calls, 5)
            nb = (4 * r * f + 4) * d
            cell["vote_median"] = {"ms_best": t["best"], "ms_median": t["median"], "coordinates_per_s": d / (t["median"] * 1e-3),
                                   "frac_of_measured_hbm": nb / (t["median"] * 1e-3) / 1e9 / peak}
            voted = torch.empty((f, d), dtype=torch.float32, device=device)
            c, m = cmax_q, f - cmax_q
            ws = bz.alloc_workspace(bz.OP_MULTIKRUM, 0, f, d, c, m, device=device)
            t = timed_calls(torch, lambda: bz.vote_multikrum(rep, c, m, voted=voted, workspace=ws, out=out), n_calls, 3)
            nb = (4 * r * f + 4 * f + 4 * m + 4) * d
            cell["vote_multikrum"] = {"ms_best": t["best"], "ms_median": t["median"], "coordinates_per_s": d / (t["median"] * 1e-3),
                                      "frac_of_measured_hbm": nb / (t["median"] * 1e-3) / 1e9 / peak,
                                      "status_bits": bz.pairdist_status(ws, f)}
            cells.append(cell)
            del rep, out, voted, ws
            torch.cuda.empty_cache()
    return {"cells": cells, "worst_case": counts,
            "note": "inputs: Gaussian file gradients, q Byzantine workers at the worst-case placement sending -100 x gradient"}


def extra_paths(bz, inputs, torch, device):
    """The other aggregators at their own configurations (not part of the headline value)."""
    res = {}
    peak, _ = measured_peaks()

    def hbm(nbytes, ms):
        gbs = nbytes / (ms * 1e-3) / 1e9
        return {"achieved_GBs": gbs, "frac_of_measured_hbm": gbs / peak}

    def timed_fp32(fn):
        """The same call with the distances kept on the binary32 kernels (the library reads the variable per call)."""
        os.environ["BZ_PAIRDIST_PATH"] = "fp32"
        try:
            return timed(torch, fn, 5, 3)
        finally:
            del os.environ["BZ_PAIRDIST_PATH"]

    # vote -> multi-Krum: K=21, r=3, l=7, f=49, d=11.2M, q=5 ALIE, c=5, m=44
    cfg = dict(MULTIKRUM)
    rep, fw, byz, cmax = make_inputs(bz, inputs, cfg, device)
    f, d, r = 49, cfg["d"], 3
    voted = torch.empty((f, d), dtype=torch.float32, device=device)
    out = torch.empty(d, dtype=torch.float32, device=device)
    ws = bz.alloc_workspace(bz.OP_MULTIKRUM, 0, f, d, 5, 44, device=device)
    sel44 = torch.arange(44, dtype=torch.int32, device=device)
    t_vote = timed(torch, lambda: bz.vote(rep, voted), 5, 3)
    ws_vw = bz.alloc_workspace(bz.OP_VOTE_VECTORWISE, r, f, d, device=device)
    t_vw = timed(torch, lambda: bz.vote_vectorwise(rep, voted, ws_vw), 5, 3)
    t_pd = timed_calls(torch, lambda: bz.pairdist(voted, ws), 10, 3)
    t_pd32 = timed_fp32(lambda: bz.pairdist(voted, ws))
    t_mean = timed(torch, lambda: bz.mean_rows(voted, sel44, out), 5, 3)
    t_mk = timed(torch, lambda: bz.multikrum(voted, 5, 44, workspace=ws, out=out), 5, 3)
    t_vm = timed(torch, lambda: bz.vote_median(rep, out), 5, 3)
    t_med = timed_calls(torch, lambda: bz.median(voted, out), 10, 3)
    t_vpd = timed(torch, lambda: bz.vote_pairdist(rep, voted, ws), 5, 3)
    t_vpd32 = timed_fp32(lambda: bz.vote_pairdist(rep, voted, ws))
    bytes_pipeline = (4 * r * f + 4 * f + 4 * f + 4 * 44 + 4) * d
    res["vote+multikrum (two calls)"] = dict(
        workload="K=21 r=3 l=7 f=49 d=11.2M, q=5 ALIE, c=5 m=44", c_max=cmax,
        coordinates_per_s=d / ((t_vote + t_mk) * 1e-3), ms_vote=t_vote, ms_multikrum=t_mk, ms_pairdist=t_pd["mean"],
        ms_pairdist_best=t_pd["best"], ms_pairdist_median=t_pd["median"],
        ms_mean_rows=t_mean, ms_pairdist_fp32=t_pd32, pairdist_fp32_fma_lane_ops_per_s=2 * (f * (f - 1) // 2) * d / (t_pd32 * 1e-3),
        pairdist=dict(kernel="integer MMA (tcgen05 kind::i8)", **hbm(4 * f * d, t_pd["median"])),
        vote=hbm((4 * r * f + 4 * f) * d, t_vote), mean_rows=hbm((4 * 44 + 4) * d, t_mean),
        pipeline=hbm(bytes_pipeline, t_vote + t_mk),
        vote_vectorwise=dict(ms=t_vw, **hbm((4 * r * f + 4 * f) * d, t_vw)),
        single_pass=dict(ms_vote_pairdist=t_vpd, ms_vote_pairdist_fp32=t_vpd32, vote_pairdist=hbm((4 * r * f + 4 * f) * d, t_vpd)))
    res["vote+median f=49"] = dict(workload="same replicas, fused vote+median", ms=t_vm, coordinates_per_s=d / (t_vm * 1e-3),
                                   **hbm((4 * r * f + 4) * d, t_vm))
    res["median f=49"] = dict(workload="median of the 49 voted rows", ms=t_med["median"], ms_best=t_med["best"],
                              coordinates_per_s=d / (t_med["median"] * 1e-3), **hbm((4 * f + 4) * d, t_med["median"]))
    del rep, voted, out, ws, ws_vw
    torch.cuda.empty_cache()

    # vote -> Bulyan: K=25, r=5, l=5, f=25, d=25M heavy-tailed, q=6 constant, c=4
    cfg = dict(BULYAN)
    rep, fw, byz, cmax = make_inputs(bz, inputs, cfg, device)
    f, d, r = 25, cfg["d"], 5
    voted = torch.empty((f, d), dtype=torch.float32, device=device)
    out = torch.empty(d, dtype=torch.float32, device=device)
    ws = bz.alloc_workspace(bz.OP_BULYAN, 0, f, d, 4, device=device)
    sel17 = torch.arange(17, dtype=torch.int32, device=device)
    t_vote = timed(torch, lambda: bz.vote(rep, voted), 5, 3)
    t_pd = timed_calls(torch, lambda: bz.pairdist(voted, ws), 10, 3)
    t_pd32 = timed_fp32(lambda: bz.pairdist(voted, ws))
    t_tm = timed_calls(torch, lambda: bz.trimmed_mean(voted, sel17, 9, out), 10, 3)
    t_bu = timed(torch, lambda: bz.bulyan(voted, 4, workspace=ws, out=out), 5, 3)
    t_vm = timed(torch, lambda: bz.vote_median(rep, out), 5, 3)
    t_vbu = timed_calls(torch, lambda: bz.vote_bulyan(rep, 4, voted=voted, workspace=ws, out=out), 10, 3)
    theta = f - 8
    bytes_pipeline = (4 * r * f + 4 * f + 4 * f + 4 * theta + 4) * d
    res["vote+bulyan"] = dict(
        workload="K=25 r=5 l=5 f=25 d=25M (1% Student-t coordinates), q=6 constant, c=4 (theta=17, beta=9)",
        c_max=cmax, coordinates_per_s=d / ((t_vote + t_bu) * 1e-3), ms_vote=t_vote, ms_bulyan=t_bu, ms_pairdist=t_pd["median"],
        ms_pairdist_best=t_pd["best"], ms_pairdist_fp32=t_pd32, ms_trimmed_mean=t_tm["median"], ms_trimmed_mean_best=t_tm["best"],
        vote=hbm((4 * r * f + 4 * f) * d, t_vote), pairdist=hbm(4 * f * d, t_pd["median"]),
        trimmed_mean=hbm((4 * theta + 4) * d, t_tm["median"]), pipeline=hbm(bytes_pipeline, t_vote + t_bu),
        single_pass=dict(ms_vote_bulyan=t_vbu["median"], ms_vote_bulyan_best=t_vbu["best"], coordinates_per_s=d / (t_vbu["median"] * 1e-3),
                         **hbm((4 * r * f + 4 * f + 4 * theta + 4) * d, t_vbu["median"])))
    res["vote+median r=5"] = dict(workload="same replicas, fused vote+median", ms=t_vm, coordinates_per_s=d / (t_vm * 1e-3),
                                  **hbm((4 * r * f + 4) * d, t_vm))
    del rep, voted, out, ws
    torch.cuda.empty_cache()

    # vote + median + model update (Eq. 1 with momentum) in one pass, headline shape
    cfg = dict(WORKLOAD)
    rep, fw, byz, cmax = make_inputs(bz, inputs, cfg, device)
    f, d, r = 25, cfg["d"], 3
    w = torch.zeros(d, dtype=torch.float32, device=device)
    vel = torch.zeros(d, dtype=torch.float32, device=device)
    out = torch.empty(d, dtype=torch.float32, device=device)
    t_fused = timed(torch, lambda: bz.vote_median_update(rep, w, 0.01, vel, 0.9), 20, 3)
    t_vm = timed(torch, lambda: bz.vote_median(rep, out), 20, 3)
    t_upd = timed(torch, lambda: bz.model_update(out, w, 0.01, vel, 0.9), 20, 3)
    res["vote+median+update"] = dict(
        workload="K=15 r=3 l=5 f=25 d=11.2M, aggregate applied to w with momentum in the same kernel",
        ms=t_fused, ms_unfused=t_vm + t_upd, coordinates_per_s=d / (t_fused * 1e-3), **hbm((4 * r * f + 16) * d, t_fused))
    del rep, w, vel, out
    torch.cuda.empty_cache()

    # exhaustive worst case: (K, f, l, r) = (35, 49, 7, 5), q = 13 - the largest row the paper printed
    _, _, mask = bz.assign_mols(7, 5)
    ws = bz.alloc_workspace(bz.OP_WORST_CASE, 5, 49)
    bz.worst_case(mask, 49, 5, 8, workspace=ws)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    cmax, arg, n = bz.worst_case(mask, 49, 5, 13, workspace=ws)
    dt = time.perf_counter() - t0
    res["worst_case"] = dict(workload="(K,f,l,r)=(35,49,7,5), q=13, all C(35,13) subsets", c_max=cmax, subsets=n,
                             seconds=dt, subsets_per_s=n / dt, argmax=[int(u) for u in arg])
    # the same maximum from one worker set per translation orbit, and the largest cluster of the sweep
    # (K = 49) up to its honest-majority limit q = 24, which the plain search cannot reach
    ws = bz.alloc_workspace(bz.OP_WORST_CASE_MOLS, 7, 49)
    bz.worst_case_mols(7, 5, 8, workspace=ws)
    sym = {}
    for l_, r_, q_ in [(7, 5, 13), (7, 7, 16), (7, 7, 24)]:
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        c_, arg_, n_ = bz.worst_case_mols(l_, r_, q_, workspace=ws)
        dt = time.perf_counter() - t0
        sym["K=%d q=%d" % (l_ * r_, q_)] = dict(c_max=c_, orbits=n_, seconds=dt, orbits_per_s=n_ / dt,
                                                argmax=[int(u) for u in arg_])
    assert sym["K=35 q=13"]["c_max"] == cmax and sym["K=35 q=13"]["argmax"] == [int(u) for u in arg]
    res["worst_case_orbits"] = sym
    return res


def profile_op(args):
    """Profiling only: run ONE entry point `--steps` times on a synthetic case of `--coords` coordinates
    (shape `--shape l,r,q`), so that a profiler capture sees just that kernel.  Prints its timing."""
    import torch

    from paper_2010_04902_b200 import binding as bz
    from paper_2010_04902_b200 import build as bz_build
    from paper_2010_04902_b200 import inputs
    bz_build.build()
    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    l, r, q = (int(x) for x in args.shape.split(","))
    f = l * l
    d = args.coords if args.coords > 0 else 2_000_000
    op = args.op
    if op == "worst_case":
        _, _, mask = bz.assign_mols(l, r)
        ws = bz.alloc_workspace(bz.OP_WORST_CASE, r, f)
        fn = lambda: bz.worst_case(mask, f, r, q, workspace=ws)
    elif op == "worst_case_mols":
        ws = bz.alloc_workspace(bz.OP_WORST_CASE_MOLS, r, f)
        fn = lambda: bz.worst_case_mols(l, r, q, workspace=ws)
    else:
        cfg = dict(l=l, r=r, q=q, d=d, attack="reversed", seed=0)
        rep, fw, byz, cmax = make_inputs(bz, inputs, cfg, device)
        voted = bz.vote(rep)
        out = torch.empty(d, dtype=torch.float32, device=device)
        c = max(0, min(cmax, (f - 3) // 4))
        ws = bz.alloc_workspace(bz.OP_MULTIKRUM, 0, f, d, c, f - c, device=device)
        theta = f - 2 * c
        sel = torch.arange(theta, dtype=torch.int32, device=device)
        sink = torch.zeros(1, dtype=torch.int64, device=device)
        fn = {
            "vote_median": lambda: bz.vote_median(rep, out),
            "vote": lambda: bz.vote(rep, voted),
            "vote_vectorwise": lambda: bz.vote_vectorwise(rep, voted),
            "median": lambda: bz.median(voted, out),
            "pairdist": lambda: bz.pairdist(voted, ws),
            "vote_pairdist": lambda: bz.vote_pairdist(rep, voted, ws),
            "vote_median_update": lambda: bz.vote_median_update(rep, out, 0.01, voted[0], 0.9),
            "multikrum": lambda: bz.multikrum(voted, c, f - c, workspace=ws, out=out),
            "vote_multikrum": lambda: bz.vote_multikrum(rep, c, f - c, voted=voted, workspace=ws, out=out),
            "vote_bulyan": lambda: bz.vote_bulyan(rep, c, voted=voted, workspace=ws, out=out),
            "bulyan": lambda: bz.bulyan(voted, c, workspace=ws, out=out),
            "mean_rows": lambda: bz.mean_rows(voted, sel, out),
            "trimmed_mean": lambda: bz.trimmed_mean(voted, sel, theta - 2 * c, out),
            "stream_probe": lambda: bz.stream_probe(rep, sink),
            "stream_probe_ring": lambda: bz.stream_probe(rep, sink, staged=True),
        }[op]
    t0 = time.perf_counter()
    ms = timed(torch, fn, args.steps, args.warmup) if not op.startswith("worst_case") else None
    if op.startswith("worst_case"):
        for _ in range(args.warmup):
            fn()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            fn()
        ms = (time.perf_counter() - t0) / args.steps * 1e3
    print(json.dumps({"profile_op": op, "shape": [l, r, q], "coordinates": d, "ms_per_call": ms}), flush=True)


def run_reference(args):
    """The CPU checker, as it stands, on the host cores: each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2010_04902_b200 import inputs
    cfg = dict(WORKLOAD)
    l, r, q = cfg["l"], cfg["r"], cfg["q"]
    f = l * l
    n_sample = 1_000_000
    wf, fw, _ = oracle.assign(l, r)
    _, byz, _ = oracle.worst_case(wf, f, r, q)
    g = inputs.true_gradients(f, n_sample, seed=cfg["seed"])
    rep = inputs.build_replicas(g, fw, byz, cfg["attack"]).numpy()
    for _ in range(args.warmup):
        oracle.vote_median(rep)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.vote_median(rep)
    dt = (time.perf_counter() - t0) / args.steps
    value = n_sample / dt
    cores = oracle.num_threads()
    sample = "first %d of %d coordinates of the same workload per step" % (n_sample, cfg["d"])
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": max(int(os.environ.get("WORLD_SIZE", "1")), int(args.gpus)),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u32", "data": "synthetic",
        "config": {"workload": workload_name(cfg), "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


def launch_ranks(n):
    """`--gpus N` without a launcher: start N ranks of this script on this node (one per GPU) and wait."""
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n), "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    os.execv(sys.executable, cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extra", action="store_true", help="skip everything but the headline, its e2e leg and the CPU baseline")
    ap.add_argument("--no-sweep", action="store_true", help="skip the (l, r) x d sweep (the longest extra leg)")
    ap.add_argument("--coords", type=int, default=0, help="profiling only: override the number of coordinates d")
    ap.add_argument("--no-e2e", action="store_true", help="profiling only: skip the host-buffer leg")
    ap.add_argument("--no-cpu", action="store_true", help="profiling only: skip the CPU baseline / parity legs")
    ap.add_argument("--op", default="", help="profiling only: run a single entry point (vote_median, vote, vote_vectorwise, median, "
                    "pairdist, vote_pairdist, vote_median_update, multikrum, vote_multikrum, bulyan, vote_bulyan, mean_rows, trimmed_mean, stream_probe, "
                    "worst_case, worst_case_mols) instead of the benchmark")
    ap.add_argument("--shape", default="5,3,3", help="profiling only: l,r,q of the cluster for --op")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.op:
        profile_op(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
            launch_ranks(args.gpus)
        if int(os.environ.get("WORLD_SIZE", "1")) != max(1, args.gpus):
            log("note: --gpus %d but the launcher started %s rank(s); the launcher's count is used"
                % (args.gpus, os.environ.get("WORLD_SIZE", "1")))
        run_ours(args)


if __name__ == "__main__":
    main()
