"""Benchmark of the ByzShield aggregation path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-extra]

One step = one fused vote + coordinate-wise median (bz_vote_median) over a resident batch of
replicated file gradients: K = 15 workers, r = 3, l = 5, f = 25 files, d = 11.2 M coordinates,
q = 3 Byzantine workers at the worst-case placement sending -100 x the true gradient.
With N > 1 (torchrun) every rank aggregates its own coordinate slab of the same size; the path needs
no collective.  Rank 0 prints ONE JSON line.  `--impl reference` times the CPU checker instead.
`--coords`, `--no-e2e`, `--no-cpu` shrink the run for profiler captures; their JSON line names the
smaller workload and is not a benchmark value.
"""
from __future__ import annotations

import argparse
import json
import os
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

# DRAM bytes per launch of the dominant kernel from an ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum, scaled to a full launch), or None when no capture of the current kernel exists.
TRAFFIC_BYTES_PER_LAUNCH = 3_420_054_000  # (600.02 + 10.70) MB at d = 2 M, scaled by 5.6 to d = 11.2 M


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
    """Samples SM clock and throttle reasons of one GPU through NVML (read-only) while a region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, torch_index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
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
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.004)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": (statistics.median(self.samples) if self.samples else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def make_inputs(bz, inputs, cfg, device, seed_offset=0, heavy=0.0):
    """Assignment and Byzantine set through the library, synthetic replicas on the device."""
    l, r, q, d = cfg["l"], cfg["r"], cfg["q"], cfg["d"]
    _, fw, mask = bz.assign_mols(l, r)
    cmax, byz, _ = bz.worst_case(mask, l * l, r, q)
    g = inputs.true_gradients(l * l, d, seed=cfg["seed"] + seed_offset, heavy_tail_frac=heavy, device=device)
    rep = inputs.build_replicas(g, fw, byz, cfg["attack"])
    del g
    return rep, fw, byz, cmax


def timed(torch, fn, steps, warmup):
    """Average device time per call in ms over `steps` calls (CUDA events on the current stream)."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


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
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    if rank == 0:
        bz_build.build()
    if world > 1:
        dist.barrier()
    bz.lib()

    cfg = dict(WORKLOAD)
    if args.coords > 0:
        cfg["d"] = args.coords
    l, r, d = cfg["l"], cfg["r"], cfg["d"]
    f = l * l
    rep, fw, byz, cmax = make_inputs(bz, inputs, cfg, device, seed_offset=rank)
    out = torch.empty(d, dtype=torch.float32, device=device)
    step = lambda: bz.vote_median(rep, out)

    # ---- timed region: exactly K steps between barriers, device time, max over ranks ----------------
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
        torch.cuda.synchronize()
    n0 = bz.kernel_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    with sampler:
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        torch.cuda.synchronize()
    launches = bz.kernel_launch_count() - n0
    if world > 1:
        dist.barrier()
    ms_total = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(ms_total, op=dist.ReduceOp.MAX)
    ms_step = float(ms_total.item()) / args.steps
    value = world * d / (ms_step * 1e-3)

    e2e, rep_host = (None, None)
    if not args.no_e2e:
        e2e, rep_host = e2e_leg(bz, torch, dist, world, rep, out, device, args.steps)

    result = None
    if rank == 0:
        peak, peak_src = measured_peaks()
        alg_bytes = (4 * r * f + 4) * d
        achieved = alg_bytes / (ms_step * 1e-3) / 1e9
        traffic = TRAFFIC_BYTES_PER_LAUNCH if args.coords == 0 else None
        result = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32",
            "data": "synthetic",
            "config": {"workload": workload_name(cfg), "coordinates_per_gpu": d, "c_max": cmax,
                       "byzantine_workers": [int(u) for u in byz],
                       "l2": "inputs are %.2f GB per step, far larger than the 126 MB L2; no flush needed" % (4 * r * f * d / 1e9),
                       "parallelism": "coordinate slabs, no collective" if world > 1 else "single GPU"},
            "clocks": sampler.summary(),
            "e2e": e2e,
            "gpu_launches": int(launches),
            "pipeline_timeouts": bz.pipeline_timeouts(),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": traffic, "peak_source": peak_src, "frac_of_nominal_8TBs": achieved / 8000.0,
                         "algorithmic_bytes_per_launch": alg_bytes,
                         "kernel": "vote_median_tma_kernel<3,25,25,3> (one launch per step)"},
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
    del rep_host, rep, out
    torch.cuda.empty_cache()

    if rank == 0 and world == 1 and not args.no_extra:
        result["other_paths"] = extra_paths(bz, inputs, torch, device)

    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(result), flush=True)


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
            return timed(torch, fn, 5, 2)
        finally:
            del os.environ["BZ_PAIRDIST_PATH"]

    # vote -> multi-Krum: K=21, r=3, l=7, f=49, d=11.2M, q=5 ALIE, c=5, m=44
    cfg = dict(l=7, r=3, q=5, d=11_200_000, attack="alie", seed=0)
    rep, fw, byz, cmax = make_inputs(bz, inputs, cfg, device)
    f, d, r = 49, cfg["d"], 3
    voted = torch.empty((f, d), dtype=torch.float32, device=device)
    out = torch.empty(d, dtype=torch.float32, device=device)
    ws = bz.alloc_workspace(bz.OP_MULTIKRUM, 0, f, d, 5, 44, device=device)
    sel44 = torch.arange(44, dtype=torch.int32, device=device)
    t_vote = timed(torch, lambda: bz.vote(rep, voted), 5, 2)
    ws_vw = bz.alloc_workspace(bz.OP_VOTE_VECTORWISE, r, f, d, device=device)
    t_vw = timed(torch, lambda: bz.vote_vectorwise(rep, voted, ws_vw), 5, 2)
    t_pd = timed(torch, lambda: bz.pairdist(voted, ws), 5, 2)
    t_pd32 = timed_fp32(lambda: bz.pairdist(voted, ws))
    t_mean = timed(torch, lambda: bz.mean_rows(voted, sel44, out), 5, 2)
    t_mk = timed(torch, lambda: bz.multikrum(voted, 5, 44, workspace=ws, out=out), 5, 2)
    t_vm = timed(torch, lambda: bz.vote_median(rep, out), 5, 2)
    t_med = timed(torch, lambda: bz.median(voted, out), 5, 2)
    t_vpd = timed(torch, lambda: bz.vote_pairdist(rep, voted, ws), 5, 2)
    t_vpd32 = timed_fp32(lambda: bz.vote_pairdist(rep, voted, ws))
    t_vmk = timed(torch, lambda: bz.vote_multikrum(rep, 5, 44, voted=voted, workspace=ws, out=out), 5, 2)
    bytes_pipeline = (4 * r * f + 4 * f + 4 * f + 4 * 44 + 4) * d
    res["vote+multikrum"] = dict(
        workload="K=21 r=3 l=7 f=49 d=11.2M, q=5 ALIE, c=5 m=44", c_max=cmax,
        coordinates_per_s=d / ((t_vote + t_mk) * 1e-3), ms_vote=t_vote, ms_multikrum=t_mk, ms_pairdist=t_pd,
        ms_mean_rows=t_mean, ms_pairdist_fp32=t_pd32, pairdist_fp32_fma_lane_ops_per_s=2 * (f * (f - 1) // 2) * d / (t_pd32 * 1e-3),
        pairdist=dict(kernel="integer MMA (tcgen05 kind::i8)", **hbm(4 * f * d, t_pd)),
        vote=hbm((4 * r * f + 4 * f) * d, t_vote), mean_rows=hbm((4 * 44 + 4) * d, t_mean),
        pipeline=hbm(bytes_pipeline, t_vote + t_mk),
        vote_vectorwise=dict(ms=t_vw, **hbm((4 * r * f + 4 * f) * d, t_vw)),
        single_pass=dict(ms_vote_pairdist=t_vpd, ms_vote_pairdist_fp32=t_vpd32, vote_pairdist=hbm((4 * r * f + 4 * f) * d, t_vpd),
                         ms_vote_multikrum=t_vmk, coordinates_per_s=d / (t_vmk * 1e-3),
                         **hbm((4 * r * f + 4 * f + 4 * 44 + 4) * d, t_vmk)))
    res["vote+median f=49"] = dict(workload="same replicas, fused vote+median", ms=t_vm, coordinates_per_s=d / (t_vm * 1e-3),
                                   **hbm((4 * r * f + 4) * d, t_vm))
    res["median f=49"] = dict(workload="median of the 49 voted rows", ms=t_med, coordinates_per_s=d / (t_med * 1e-3),
                              **hbm((4 * f + 4) * d, t_med))
    del rep, voted, out, ws
    torch.cuda.empty_cache()

    # vote -> Bulyan: K=25, r=5, l=5, f=25, d=25M heavy-tailed, q=6 constant, c=4
    cfg = dict(l=5, r=5, q=6, d=25_000_000, attack="constant", seed=0)
    rep, fw, byz, cmax = make_inputs(bz, inputs, cfg, device, heavy=0.01)
    f, d, r = 25, cfg["d"], 5
    voted = torch.empty((f, d), dtype=torch.float32, device=device)
    out = torch.empty(d, dtype=torch.float32, device=device)
    ws = bz.alloc_workspace(bz.OP_BULYAN, 0, f, d, 4, device=device)
    sel17 = torch.arange(17, dtype=torch.int32, device=device)
    t_vote = timed(torch, lambda: bz.vote(rep, voted), 5, 2)
    t_pd = timed(torch, lambda: bz.pairdist(voted, ws), 5, 2)
    t_pd32 = timed_fp32(lambda: bz.pairdist(voted, ws))
    t_tm = timed(torch, lambda: bz.trimmed_mean(voted, sel17, 9, out), 5, 2)
    t_bu = timed(torch, lambda: bz.bulyan(voted, 4, workspace=ws, out=out), 5, 2)
    t_vm = timed(torch, lambda: bz.vote_median(rep, out), 5, 2)
    t_vbu = timed(torch, lambda: bz.vote_bulyan(rep, 4, voted=voted, workspace=ws, out=out), 5, 2)
    theta = f - 8
    bytes_pipeline = (4 * r * f + 4 * f + 4 * f + 4 * theta + 4) * d
    res["vote+bulyan"] = dict(
        workload="K=25 r=5 l=5 f=25 d=25M (1% Student-t coordinates), q=6 constant, c=4 (theta=17, beta=9)",
        c_max=cmax, coordinates_per_s=d / ((t_vote + t_bu) * 1e-3), ms_vote=t_vote, ms_bulyan=t_bu, ms_pairdist=t_pd,
        ms_pairdist_fp32=t_pd32, ms_trimmed_mean=t_tm, vote=hbm((4 * r * f + 4 * f) * d, t_vote), pairdist=hbm(4 * f * d, t_pd),
        trimmed_mean=hbm((4 * theta + 4) * d, t_tm), pipeline=hbm(bytes_pipeline, t_vote + t_bu),
        single_pass=dict(ms_vote_bulyan=t_vbu, coordinates_per_s=d / (t_vbu * 1e-3),
                         **hbm((4 * r * f + 4 * f + 4 * theta + 4) * d, t_vbu)))
    res["vote+median r=5"] = dict(workload="same replicas, fused vote+median", ms=t_vm, coordinates_per_s=d / (t_vm * 1e-3),
                                  **hbm((4 * r * f + 4) * d, t_vm))
    del rep, voted, out, ws
    torch.cuda.empty_cache()

    # vote + median + model update (Eq. 1 with momentum) in one pass, headline shape
    cfg = dict(l=5, r=3, q=3, d=11_200_000, attack="reversed", seed=0)
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
        fn = {
            "vote_median": lambda: bz.vote_median(rep, out),
            "vote": lambda: bz.vote(rep, voted),
            "vote_vectorwise": lambda: bz.vote_vectorwise(rep, voted),
            "median": lambda: bz.median(voted, out),
            "pairdist": lambda: bz.pairdist(voted, ws),
            "vote_pairdist": lambda: bz.vote_pairdist(rep, voted, ws),
            "vote_median_update": lambda: bz.vote_median_update(rep, out, 0.01, voted[0], 0.9),
            "multikrum": lambda: bz.multikrum(voted, c, f - c, workspace=ws, out=out),
            "bulyan": lambda: bz.bulyan(voted, c, workspace=ws, out=out),
            "mean_rows": lambda: bz.mean_rows(voted, sel, out),
            "trimmed_mean": lambda: bz.trimmed_mean(voted, sel, theta - 2 * c, out),
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
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u32", "data": "synthetic",
        "config": {"workload": workload_name(cfg), "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extra", action="store_true", help="skip the multi-Krum / Bulyan / worst-case extras")
    ap.add_argument("--coords", type=int, default=0, help="profiling only: override the number of coordinates d")
    ap.add_argument("--no-e2e", action="store_true", help="profiling only: skip the host-buffer leg")
    ap.add_argument("--no-cpu", action="store_true", help="profiling only: skip the CPU baseline / parity leg")
    ap.add_argument("--op", default="", help="profiling only: run a single entry point (vote_median, vote, vote_vectorwise, median, "
                    "pairdist, vote_pairdist, vote_median_update, multikrum, bulyan, mean_rows, trimmed_mean, worst_case, "
                    "worst_case_mols) instead of the benchmark")
    ap.add_argument("--shape", default="5,3,3", help="profiling only: l,r,q of the cluster for --op")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.op:
        profile_op(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
