#!/usr/bin/env python
"""Benchmark of the EMC2 data bridge + dispatch on B200.

A step is one pass of the whole hot path (emc2_bridge_run: voxelize, project +
gather, route + dispatch; the three stage calls back to back are timed as well)
over one batch of synthetic frames.  Default workload: the nuScenes-shaped 6-camera batch (4 frames of
300,000 points), the configuration the roofline target is quoted on.

    python bench.py --gpus 1 --steps 20 --warmup 5
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N   (replicas, weak scaling)
    python bench.py --impl reference      (the CPU oracle on the host cores)
    python bench.py --config 1            (another workload; --sweep for the throughput grid)

Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import emc2_gen as gen

NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126e6


# ----------------------------------------------------------------------------- helpers
def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes(w, B, N, m0, m1, texels):
    """Bytes the staged ABI must move: every input read once per call, every output written once."""
    pb, fb, C = 4 * w.C, 4 * w.feat_c, w.C
    g1 = w.grids[1]
    vox = B * N * pb + B * N * 8 + (m0 + m1) * (16 + 4 + pb) + B * C * g1.dims[1] * g1.dims[0] * 4
    pg = B * N * pb + B * w.K * 48 + fb * texels + B * N * (12 + 1 + 1 + fb)
    rd = B * N * (pb + 1 + fb) + B * N * (1 + 4 + pb + fb) + B * (w.num_experts + 1) * 4
    return {"voxelize": vox, "project_gather": pg, "route_dispatch": rd, "total": vox + pg + rd}


def kernel_bytes(w, B, N, texels):
    """Algorithmic bytes of the row-moving kernels, per launch."""
    pb, fb = 4 * w.C, 4 * w.feat_c
    return {"project_gather": B * N * pb + B * w.K * 48 + fb * texels + B * N * (12 + 1 + 1 + fb),
            "dispatch_scatter": B * N * (1 + pb + fb) + B * N * (4 + pb + fb),
            # one-call path: reads points, uvd, camera, expert and the texels; writes the permutation,
            # the point rows and every feature row twice (gathered and feat_out)
            "gather_scatter": B * N * (pb + 12 + 1 + 1) + fb * texels + B * N * (4 + pb + 2 * fb)}


def one_call_bytes(w, B, N, m0, m1, texels):
    """Bytes the one-call path must move: as the staged count, minus the read-back of `gathered`,
    of the mask and of the point rows that stages 3 - 4 no longer need, plus the re-read of uvd/cam."""
    pb, fb = 4 * w.C, 4 * w.feat_c
    staged = algorithmic_bytes(w, B, N, m0, m1, texels)
    proj = B * N * pb + B * w.K * 48 + B * N * (12 + 1 + 1 + 1)
    return staged["voxelize"] + proj + kernel_bytes(w, B, N, texels)["gather_scatter"] + B * (w.num_experts + 1) * 4


def bridge_fractions(own_bytes, staged_bytes, ms_step, staged_ms, peak, peak_kind):
    """The bandwidth figures of the bench line.  Every time is paired with the bytes that path moves: the
    one-call step with the one-call byte count (the headline), the three stage calls with the staged count.
    The staged count over the one-call time is kept under a name that says what it is."""
    own_gbs = own_bytes / (ms_step * 1e-3) / 1e9
    staged_gbs = staged_bytes / (staged_ms * 1e-3) / 1e9
    equiv_gbs = staged_bytes / (ms_step * 1e-3) / 1e9
    return {
        "one_call_bytes_per_step": own_bytes,
        "bridge_own_gbs": own_gbs,
        "bridge_frac_of_8tbs_own_bytes": own_gbs / NOMINAL_HBM_GBS,
        f"bridge_frac_of_{peak_kind}_copy_own_bytes": own_gbs / peak,
        "target_50pct_of_8tbs_met": bool(own_gbs / NOMINAL_HBM_GBS >= 0.5),
        "staged_path": {"ms_per_step": staged_ms, "gbs": staged_gbs, "frac_of_8tbs": staged_gbs / NOMINAL_HBM_GBS,
                        f"frac_of_{peak_kind}_copy": staged_gbs / peak},
        "equivalent_staged_bandwidth": {"gbs": equiv_gbs, "frac_of_8tbs": equiv_gbs / NOMINAL_HBM_GBS,
                                        "note": "bytes of the three stage calls divided by the one-call time; "
                                                "the one-call path does not move all of them"},
    }


def distinct_texels(w, pg):
    """Distinct feature texels the gather touches, from the library's own uvd/cam outputs."""
    uvd, cam = pg["uvd"], pg["cam"]
    B, N = cam.shape
    vis = cam >= 0
    off = float(getattr(w, "feat_offset", 0.0))
    fx = ((uvd[..., 0] - off) / w.feat_stride)[vis]
    fy = ((uvd[..., 1] - off) / w.feat_stride)[vis]
    b = torch.arange(B, device=cam.device)[:, None].expand(B, N)[vis].long()
    k = cam[vis].long()
    x0, y0 = fx.floor().long(), fy.floor().long()
    keys = []
    for dy in (0, 1):
        for dx in (0, 1):
            x = (x0 + dx).clamp(min=0, max=w.feat_w - 1)
            y = (y0 + dy).clamp(min=0, max=w.feat_h - 1)
            keys.append(((b * w.K + k) * w.feat_h + y) * w.feat_w + x)
    return int(torch.unique(torch.cat(keys)).numel())


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "100", "-i", str(index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            out = {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                   "samples": len(sm)}
        return out


def source_digest():
    """SHA-256 over the CUDA sources and internal headers: ncu counters are valid for the code they were taken on."""
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2507_04123_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        if name.endswith((".cu", ".cuh")):
            with open(os.path.join(csrc, name), "rb") as f:
                h.update(name.encode() + b"\0" + f.read())
    return h.hexdigest()[:16]


def make_bridge(pkg, w, device, tune):
    br = pkg.Bridge(pkg.config_from_workload(w, device=device))
    for k, v in tune:
        br.set_tuning(k, v)
    return br


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


# ----------------------------------------------------------------------------- reference arm (CPU oracle)
def oracle_rate(w, target_s=12.0, max_steps=None, points=None):
    """Times the oracle, as it stands, single-threaded on the host, on one-frame samples."""
    import oracle
    oracle.build()
    w1 = w.with_shape(1, points or w.N)
    batch = gen.make_batch(w1, frames=[0])
    oracle.bridge(w1, batch)                               # warm the caches / page in
    times = []
    t_all = time.perf_counter()
    while True:
        t0 = time.perf_counter()
        oracle.bridge(w1, batch)
        times.append(time.perf_counter() - t0)
        if max_steps is not None and len(times) >= max_steps:
            break
        if max_steps is None and time.perf_counter() - t_all > target_s and len(times) >= 3:
            break
    return times


def run_reference(args, w):
    rank, _, world = dist_env()
    if rank != 0:
        return
    steps = args.steps
    # A step is one frame through the oracle; with many steps the frame is cut to its first points so
    # that the whole run stays near two minutes (the oracle costs about 0.9 us per point).
    budget_points = int(120.0 / (steps + args.warmup) / 0.9e-6)
    n = max(1024, min(w.N, budget_points))
    times = oracle_rate(w, max_steps=args.warmup + steps, points=n)[args.warmup:]
    per = float(np.median(times))
    fps = (n / per) / w.N                                  # frames of the full size per second
    sample = (f"1 frame of {n} of {w.N} points per step, median of {steps} steps"
              + ("" if n == w.N else "; frames/s scaled by points"))
    line = {
        "impl": "reference", "metric": "bridge frames/s", "value": fps, "unit": "frames/s",
        "n_gpus": args.gpus, "steps": steps, "warmup": args.warmup, "ms_per_step": per * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "points_per_frame": w.N, "cameras": w.K, "feat_c": w.feat_c,
                   "step": "one frame through the single-threaded C++ oracle"},
        "mpoints_per_s": n / per / 1e6,
        "cpu_baseline": {"value": fps, "unit": "frames/s", "cores": 1, "kind": "oracle", "sample": sample,
                         "host_cores_available": os.cpu_count()},
        "e2e": {"value": fps, "unit": "frames/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- our arm
def time_steps(fn, steps, stream_sync, barrier):
    barrier()
    stream_sync()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        fn()
    b.record()
    stream_sync()
    barrier()
    return a.elapsed_time(b) / 1e3


def run_ours(args, w):
    import paper_2507_04123_b200 as pkg
    from paper_2507_04123_b200 import build as cuda_build
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the bridge has no CPU path")
    if not os.path.exists(pkg.LIB_PATH):
        cuda_build.build()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    use_dist = world > 1
    if use_dist:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if use_dist:
            dist.barrier()

    from paper_2507_04123_b200 import sharding

    def max_over_ranks(x):
        return sharding.max_over_ranks(x, dev)

    B, N = w.B, w.N
    frames = sharding.frames_for_rank(rank, world, B)      # every rank owns its own frames
    batch = gen.make_batch(w, frames=frames, feature_frames=args.feature_frames)
    if args.point_order == "azimuth":
        # Context only: the generators shuffle the points of a frame; a spinning LiDAR delivers them in
        # firing order.  Sorting by azimuth (then range) stands in for that.
        pts = batch["points"]
        for b in range(pts.shape[0]):
            key = np.lexsort((np.hypot(pts[b, :, 0], pts[b, :, 1]), np.arctan2(pts[b, :, 1], pts[b, :, 0])))
            pts[b] = pts[b][key]
    host = {k: torch.from_numpy(v).pin_memory() for k, v in batch.items()}
    d = {k: v.to(dev, non_blocking=True) for k, v in host.items()}
    sync = lambda: torch.cuda.synchronize(dev)
    pool_info = None
    if args.pool > 1:
        # Multiscale Pooling first (its own kernel, timed alone), then the bridge on the pooled maps.
        from dataclasses import replace
        br0 = make_bridge(pkg, w, local_rank, args.tune)
        pooled = br0.pool_features(d["feat"], args.pool)
        for _ in range(3):
            br0.pool_features(d["feat"], args.pool, out=pooled)
        secs_pool = time_steps(lambda: br0.pool_features(d["feat"], args.pool, out=pooled), args.steps, sync, barrier)
        br0.status()
        br0.close()
        pbytes = d["feat"].numel() * 4 + pooled.numel() * 4
        peak0, kind0 = measured_peak()
        gbs = pbytes / (secs_pool / args.steps) / 1e9
        pool_info = {"p": args.pool, "ms_per_launch": secs_pool / args.steps * 1e3, "bytes_per_launch": pbytes,
                     "achieved_gbs": gbs, f"frac_of_{kind0}_copy": gbs / peak0}
        unpooled = (w, d["feat"])
        w = replace(w, name=f"{w.name}_pool{args.pool}", feat_stride=w.feat_stride * args.pool,
                    feat_offset=(args.pool - 1) / 2 * w.feat_stride)
        d["feat"] = pooled
        host["feat"] = pooled.cpu().pin_memory()
    br = make_bridge(pkg, w, local_rank, args.tune)

    bufs = br.run(d["points"], d["proj"], d["feat"])
    br.status()
    nv = bufs["vox"]["num_voxels"].cpu().numpy()
    texels = distinct_texels(w, bufs["pg"])
    abytes = algorithmic_bytes(w, B, N, int(nv[0]), int(nv[1]), texels)

    def step():                                            # emc2_bridge_run: the whole path in one call
        br.run(d["points"], d["proj"], d["feat"], bufs)

    def staged_step():                                     # the same work as three stage calls
        br.run_staged(d["points"], d["proj"], d["feat"], bufs)

    for _ in range(max(args.warmup, 3)):
        step()
    sync()
    br.profile_read(reset=True)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        time.sleep(0.3)
    # The timed region is exactly `steps` steps between barriers and synchronisations; it is taken
    # `repeats` times and the median region is reported (a 20-step region lasts a few milliseconds).
    regions = [max_over_ranks(time_steps(step, args.steps, sync, barrier)) for _ in range(max(1, args.repeats))]
    secs = float(np.median(regions))
    launches = sum(n for n, _ in br.profile_read(reset=True).values()) // max(1, args.repeats)
    br.status()
    for _ in range(3):
        staged_step()
    staged_secs = max_over_ranks(time_steps(staged_step, args.steps, sync, barrier))
    dispatch_only_secs = None
    if args.dispatch_only:
        # The same call for a consumer of the dispatched rows only: the rows in point order are not stored.
        kept = bufs["pg"]["gathered"]
        bufs["pg"]["gathered"] = None
        for _ in range(args.warmup):
            step()
        dispatch_only_secs = max_over_ranks(time_steps(step, args.steps, sync, barrier))
        br.status()
        bufs["pg"]["gathered"] = kept
        step()
    graph_secs = None
    if args.graph:
        # The one-call step captured once into a CUDA graph and replayed (fewer launch gaps on small batches).
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        for _ in range(args.warmup):
            graph.replay()
        graph_secs = max_over_ranks(time_steps(graph.replay, args.steps, sync, barrier))
        br.status()
    br.profile_read(reset=True)

    # End to end through the host-buffer entry point (emc2_bridge_run_host): every step copies its inputs
    # in from pinned host memory and its small results back.  Two handles, streams and buffer sets take
    # the steps in turn, so the copies of one step run beside the kernels of the other.
    e2e_secs = None
    e2e_steps = max(4, min(args.steps, 20))
    if not args.no_e2e:
        lanes = []
        for i in range(2):
            lane = {"br": br if i == 0 else make_bridge(pkg, w, local_rank, args.tune),
                    "stream": torch.cuda.Stream(device=dev),
                    "staging": {k: torch.empty_like(v) for k, v in d.items()},
                    "off": torch.empty((B, w.num_experts + 1), dtype=torch.int32).pin_memory(),
                    "nv": torch.empty((2,), dtype=torch.int32).pin_memory()}
            lane["bufs"] = bufs if i == 0 else lane["br"].run(d["points"], d["proj"], d["feat"])
            lanes.append(lane)
        sync()
        e2e_count = [0]

        def e2e_step():
            lane = lanes[e2e_count[0] & 1]
            e2e_count[0] += 1
            with torch.cuda.stream(lane["stream"]):
                lane["br"].run_host(host, lane["staging"], lane["bufs"], lane["off"], lane["nv"])

        def e2e_time():
            # Events on the timing stream see the lanes' streams through joins on both sides.
            main = torch.cuda.current_stream(dev)
            barrier()
            sync()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record(main)
            for lane in lanes:
                lane["stream"].wait_event(t0)
            for _ in range(e2e_steps):
                e2e_step()
            for lane in lanes:
                done = torch.cuda.Event()
                done.record(lane["stream"])
                main.wait_event(done)
            t1.record(main)
            sync()
            barrier()
            return t0.elapsed_time(t1) / 1e3

        for _ in range(4):
            e2e_step()
        sync()
        e2e_secs = max_over_ranks(e2e_time())
        for lane in lanes:
            lane["br"].status()
        assert torch.equal(lanes[1]["off"], bufs["rd"]["offsets"].cpu())
        lanes[1]["br"].close()
    clocks = sampler.stop() if sampler else None
    h2d = sum(int(host[k].numel() * host[k].element_size()) for k in ("points", "proj", "feat"))
    d2h = int(B * (w.num_experts + 1) * 4 + 2 * 4)

    # Per-kernel device time (events around every launch), outside the timed region.
    br.profile_read(reset=True)
    br.profile_enable(True)
    prof_steps = max(3, min(args.steps, 10))
    br.set_overlap(False)                                  # kernels one after another: clean per-kernel times
    for _ in range(prof_steps):
        step()
    sync()
    br.set_overlap(True)
    sync()
    prof = br.profile_read(reset=True)
    br.profile_enable(False)
    kb = kernel_bytes(w, B, N, texels)
    per_kernel = {k: {"launches": n, "ms_per_launch": (ms / n if n else 0.0)} for k, (n, ms) in prof.items() if n}
    dom = max((k for k in per_kernel if k in kb), key=lambda k: per_kernel[k]["ms_per_launch"] * per_kernel[k]["launches"])
    peak, peak_kind = measured_peak()
    dom_ms = per_kernel[dom]["ms_per_launch"]
    achieved = kb[dom] / (dom_ms * 1e-3) / 1e9 if dom_ms > 0 else 0.0
    traffic, traffic_stale = None, None
    try:                                                   # ncu DRAM counters, taken on this workload only
        if w.config_id == 2 and args.pool <= 1 and not args.batch and not args.points and not args.tune:
            with open(os.path.join(ROOT, "profiles", "dram_traffic_nuscenes.json")) as f:
                tj = json.load(f)
            t = tj.get("kernels", {}).get(dom)
            # counters are valid for the sources they were taken on: otherwise the figure is withheld
            traffic_stale = tj.get("source_digest") != source_digest()
            if t and not traffic_stale:
                traffic = t["dram_bytes_per_point"] * B * N
    except Exception:
        pass

    timeline = None
    if args.timeline:
        # One step with both streams on, every launch bracketed by events: who ran beside whom.
        br.profile_read(reset=True)
        br.profile_enable(True)
        for _ in range(3):
            step()
            sync()
            timeline = br.profile_timeline()
        br.profile_enable(False)

    if rank != 0:
        if use_dist:
            dist.destroy_process_group()
        return

    ms_step = secs / args.steps * 1e3
    fps = world * B * args.steps / secs
    own_bytes = one_call_bytes(w, B, N, int(nv[0]), int(nv[1]), texels)
    staged_ms = staged_secs / args.steps * 1e3
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        times = oracle_rate(w, target_s=12.0)
        per = float(np.median(times))
        cpu = {"value": 1.0 / per, "unit": "frames/s", "cores": 1, "kind": "oracle",
               "sample": f"{len(times)} single-frame passes ({w.N} points each), median; host has {os.cpu_count()} cores",
               "ms_per_frame": per * 1e3}
    line = {
        "metric": "bridge frames/s", "value": fps, "unit": "frames/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "frames_per_step_per_gpu": B, "points_per_frame": N, "point_floats": w.C,
                   "cameras": w.K, "feat_c": w.feat_c, "point_order": args.point_order,
                   "parallelism": f"replicas x{world} (frames sharded, no collective)",
                   "l2": "inputs and outputs of a step exceed L2 (no flush)" if abytes["total"] > 2 * L2_BYTES
                         else "working set fits in L2 (latency-bound workload, no flush)"},
        "mpoints_per_s": fps * N / 1e6,
        "staged_ms_per_step": staged_secs / args.steps * 1e3,
        "dispatch_only_ms_per_step": dispatch_only_secs / args.steps * 1e3 if dispatch_only_secs is not None else None,
        "graph_ms_per_step": graph_secs / args.steps * 1e3 if graph_secs is not None else None,
        "repeats": {"regions": len(regions), "ms_per_step_min": min(regions) / args.steps * 1e3,
                    "ms_per_step_median": ms_step, "ms_per_step_max": max(regions) / args.steps * 1e3},
        **bridge_fractions(own_bytes, abytes["total"], ms_step, staged_ms, peak, peak_kind),
        "bridge_algorithmic_bytes_per_step": abytes,
        "roofline": {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "peak_source": peak_kind,
                     "unit": "GB/s", "frac": achieved / peak, "traffic": traffic, "traffic_stale": traffic_stale,
                     "algorithmic_bytes_per_launch": kb[dom], "ms_per_launch": dom_ms},
        "kernels": per_kernel,
        "e2e": {"value": world * B * e2e_steps / e2e_secs, "unit": "frames/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_secs / e2e_steps * 1e3,
                "call": "emc2_bridge_run_host; two handles and streams take the steps in turn, so one step's copies run "
                        "beside the other's kernels"}
        if e2e_secs else None,
        "gpu_launches": launches, "clocks": clocks, "cpu_baseline": cpu,
        "unique_voxels": [int(nv[0]), int(nv[1])], "distinct_texels": texels,
    }
    if w.config_id == 2 and world == 1 and not args.no_other_workloads and args.pool <= 1 and not args.batch \
            and not args.points:
        # The KITTI-shaped batch and the dense frame, briefly (same call, same tuning), so that their numbers
        # are in the same record as the headline workload's.
        line["other_workloads"] = {gen.workload(c).name: short_run(pkg, gen.workload(c), local_rank, args.tune)
                                   for c in (1, 3)}
    if args.tune:
        line["tuning"] = {k: v for k, v in args.tune}
    if timeline:
        line["timeline_ms"] = [{"kernel": k, "start": round(a, 4), "end": round(b, 4)} for k, a, b in timeline]
    if pool_info:
        line["multiscale_pooling"] = pool_info
    if args.occlusion:
        # Depth-buffer occlusion on the step's visibility mask (three kernels, timed together).
        cell = w.feat_stride
        occ = br.occlusion(d["points"], d["proj"], bufs["pg"]["vis_mask"], cell, 0.5)
        fn = lambda: br.occlusion(d["points"], d["proj"], bufs["pg"]["vis_mask"], cell, 0.5, occ)
        for _ in range(3):
            fn()
        secs_oc = time_steps(fn, args.steps, sync, barrier)
        br.status()
        obytes = 2 * B * N * (4 * w.C + 1) + occ["zbuf"].numel() * 4 + 2 * B * N
        ms_oc = secs_oc / args.steps * 1e3
        line["occlusion"] = {"cell_px": cell, "margin_m": 0.5, "ms_per_call": ms_oc, "algorithmic_bytes": obytes,
                             "achieved_gbs": obytes / (ms_oc * 1e-3) / 1e9,
                             "occluded_share_of_visible": float((occ["occ_mask"] != 0).sum().item())
                             / max(1.0, float((bufs["pg"]["vis_mask"] != 0).sum().item()))}
    if args.voxel_image:
        # Fusion by voxel on the outputs of the step, per scale (three kernels each, timed together).
        vi = {}
        pg = bufs["pg"]
        for sc in (0, 1):
            out = br.voxel_image(bufs["vox"], sc, pg["vis_mask"], pg["gathered"])
            fn = lambda: br.voxel_image(bufs["vox"], sc, pg["vis_mask"], pg["gathered"], out)
            for _ in range(3):
                fn()
            secs_vi = time_steps(fn, args.steps, sync, barrier)
            br.status()
            M = int(nv[sc])
            nvis = int(out["vox_img_count"][:M].sum().item())
            vbytes = B * N * 5 + M * 4 + nvis * 4 * w.feat_c + M * (4 * w.feat_c + 4)
            ms_vi = secs_vi / args.steps * 1e3
            # the same rows blended straight from the maps (no per-point rows read): the tap bytes are served
            # from L2 mostly, so the algorithmic bytes are the lists, 13 B per point and the voxel rows
            fn2 = lambda: br.voxel_image_sampled(bufs["vox"], sc, pg["uvd"], pg["cam"], d["feat"], out)
            for _ in range(3):
                fn2()
            secs_vs = time_steps(fn2, args.steps, sync, barrier)
            br.status()
            ms_vs = secs_vs / args.steps * 1e3
            sbytes = B * N * 4 + M * 4 + nvis * 13 + texels * 4 * w.feat_c + M * (4 * w.feat_c + 4)
            fused = {}
            if args.pool > 1:
                # Multiscale Pooling folded into the per-voxel sampling (window means taken where the taps are
                # read, from the unpooled maps) against pooling first and sampling the pooled maps.
                w0, feat0 = unpooled
                br_u = make_bridge(pkg, w0, local_rank, args.tune)
                fn3 = lambda: br_u.voxel_image_pooled(bufs["vox"], sc, pg["uvd"], pg["cam"], feat0, args.pool, out)
                for _ in range(3):
                    fn3()
                secs_vp = time_steps(fn3, args.steps, sync, barrier)
                br_u.status()
                br_u.close()
                fused = {"pooling_folded_into_sampling_ms_per_call": secs_vp / args.steps * 1e3,
                         "pool_then_sample_ms": pool_info["ms_per_launch"] + ms_vs}
            vi[f"scale{sc}"] = {**fused, "ms_per_call": ms_vi, "voxels": M, "visible_points": nvis,
                                "algorithmic_bytes": vbytes, "achieved_gbs": vbytes / (ms_vi * 1e-3) / 1e9,
                                "sampled_ms_per_call": ms_vs, "sampled_algorithmic_bytes": sbytes,
                                "sampled_achieved_gbs": sbytes / (ms_vs * 1e-3) / 1e9}
        line["voxel_image"] = vi
    if args.rulebook:
        # Sparse-convolution rulebook of each scale's voxel list (five kernels, timed together).
        rb = {}
        for sc in (0, 1):
            M = int(nv[sc])
            out = br.rulebook(bufs["vox"], sc)
            fn = lambda: br.rulebook(bufs["vox"], sc, out=out)
            for _ in range(3):
                fn()
            secs_rb = time_steps(fn, args.steps, sync, barrier)
            br.status()
            br.profile_read(reset=True)
            br.profile_enable(True)
            for _ in range(5):
                fn()
            sync()
            kern = {k: ms / n for k, (n, ms) in br.profile_read(reset=True).items() if n and k.startswith("rb_")}
            br.profile_enable(False)
            pairs = int(out["offsets"][27].item())
            rbytes = 16 * M + 8 * pairs + 112            # the list read once, every pair written once
            ms_rb = secs_rb / args.steps * 1e3
            rb[f"scale{sc}"] = {"ms_per_call": ms_rb, "voxels": M, "pairs": pairs, "algorithmic_bytes": rbytes,
                                "achieved_gbs": rbytes / (ms_rb * 1e-3) / 1e9,
                                "pairs_per_s": pairs / (ms_rb * 1e-3), "kernel_ms": kern}
        line["rulebook"] = rb
    if args.channels_last:
        # Planar maps -> channels-last, its own kernel timed alone (a pure copy: bytes = 2 x the maps).
        planar = d["feat"].permute(0, 1, 4, 2, 3).contiguous()
        cl = br.features_channels_last(planar)
        assert torch.equal(cl, d["feat"])
        fn = lambda: br.features_channels_last(planar, cl)
        for _ in range(3):
            fn()
        secs_cl = time_steps(fn, args.steps, sync, barrier)
        br.status()
        cbytes = 2 * planar.numel() * 4
        ms_cl = secs_cl / args.steps * 1e3
        peak1, kind1 = measured_peak()
        line["channels_last"] = {"ms_per_call": ms_cl, "algorithmic_bytes": cbytes,
                                 "achieved_gbs": cbytes / (ms_cl * 1e-3) / 1e9,
                                 f"frac_of_{kind1}_copy": cbytes / (ms_cl * 1e-3) / 1e9 / peak1}
    print(json.dumps(line), flush=True)
    if use_dist:
        dist.destroy_process_group()


def short_run(pkg, w, device, tune, steps=20, repeats=3):
    """One-call step time and own-byte fraction of another workload (no staged, host-buffer or CPU legs)."""
    dev = torch.device("cuda", device)
    batch = gen.make_batch(w)
    d = {k: torch.from_numpy(v).to(dev) for k, v in batch.items()}
    br = make_bridge(pkg, w, device, tune)
    bufs = br.run(d["points"], d["proj"], d["feat"])
    br.status()
    nv = bufs["vox"]["num_voxels"].cpu().numpy()
    own = one_call_bytes(w, w.B, w.N, int(nv[0]), int(nv[1]), distinct_texels(w, bufs["pg"]))
    step = lambda: br.run(d["points"], d["proj"], d["feat"], bufs)
    for _ in range(5):
        step()
    sync = lambda: torch.cuda.synchronize(dev)
    regions = [time_steps(step, steps, sync, lambda: None) for _ in range(repeats)]
    br.status()
    br.close()
    ms = float(np.median(regions)) / steps * 1e3
    gbs = own / (ms * 1e-3) / 1e9
    return {"frames_per_step": w.B, "points_per_frame": w.N, "ms_per_step": ms, "frames_per_s": w.B / (ms * 1e-3),
            "mpoints_per_s": w.B * w.N / (ms * 1e-3) / 1e6, "one_call_bytes_per_step": own, "own_gbs": gbs,
            "frac_of_8tbs_own_bytes": gbs / NOMINAL_HBM_GBS, "steps": steps, "regions": repeats}


def run_sweep(args):
    """Throughput grid: points per frame x batch through the six-camera projection (1 GPU)."""
    import paper_2507_04123_b200 as pkg
    dev = torch.device("cuda", 0)
    rows = []
    for N in gen.SWEEP_POINTS:
        for B in gen.SWEEP_BATCH:
            w = gen.SWEEP.with_shape(B, N)
            batch = gen.make_batch(w, feature_frames=1)
            d = {k: torch.from_numpy(v).to(dev) for k, v in batch.items()}
            br = pkg.Bridge(pkg.config_from_workload(w))
            bufs = br.run(d["points"], d["proj"], d["feat"])
            br.status()
            nv = bufs["vox"]["num_voxels"].cpu().numpy()
            tex = distinct_texels(w, bufs["pg"])
            ab = algorithmic_bytes(w, B, N, int(nv[0]), int(nv[1]), tex)
            own = one_call_bytes(w, B, N, int(nv[0]), int(nv[1]), tex)
            step = lambda: br.run(d["points"], d["proj"], d["feat"], bufs)
            for _ in range(5):
                step()
            steps = 20 if B * N < 4_000_000 else 8
            secs = time_steps(step, steps, lambda: torch.cuda.synchronize(dev), lambda: None)
            ms = secs / steps * 1e3
            gbs = own / (ms * 1e-3) / 1e9                   # the bytes the one-call path moves over its time
            rows.append({"N": N, "B": B, "ms_per_step": ms, "frames_per_s": B / (ms * 1e-3),
                         "mpoints_per_s": B * N / (ms * 1e-3) / 1e6, "own_gbs": gbs,
                         "frac_of_8tbs_own_bytes": gbs / NOMINAL_HBM_GBS, "own_bytes_per_point": own / (B * N),
                         "staged_bytes_per_point": ab["total"] / (B * N)})
            br.close()
            del d, bufs
            torch.cuda.empty_cache()
            print(json.dumps(rows[-1]), flush=True)
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="workload id 0..3 (default: nuScenes-shaped)")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--points", type=int, default=None)
    ap.add_argument("--feature-frames", type=int, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--sweep", action="store_true")
    ap.add_argument("--occlusion", action="store_true", help="also time emc2_occlusion (depth-buffer test)")
    ap.add_argument("--point-order", choices=["shuffled", "azimuth"], default="shuffled",
                    help="order of the points inside a frame (default: the generators' shuffled order)")
    ap.add_argument("--dispatch-only", action="store_true",
                    help="also time the one-call step without the feature rows in point order (d_gathered = NULL)")
    ap.add_argument("--graph", action="store_true", help="also time the one-call step replayed from a CUDA graph")
    ap.add_argument("--rulebook", action="store_true", help="also time emc2_rulebook (sparse-convolution rulebook)")
    ap.add_argument("--channels-last", action="store_true", help="also time emc2_features_channels_last")
    ap.add_argument("--voxel-image", action="store_true", help="also time emc2_voxel_image (fusion by voxel)")
    ap.add_argument("--repeats", type=int, default=5, help="timed regions of --steps steps each; the median is reported")
    ap.add_argument("--tune", action="append", default=[], metavar="KNOB=VALUE",
                    help="emc2_bridge_set_tuning on every handle (row_store)")
    ap.add_argument("--timeline", action="store_true", help="add one step's per-launch start/end times on both streams")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the short runs of the KITTI-shaped and dense workloads")
    ap.add_argument("--pool", type=int, default=1, help="Multiscale Pooling size p (power of two): pool the maps, "
                                                        "then run the bridge on the pooled maps")
    args = ap.parse_args()
    args.tune = [(kv.split("=")[0], int(kv.split("=")[1])) for kv in args.tune]
    w = gen.workload(args.config)
    if args.batch or args.points:
        w = w.with_shape(args.batch or w.B, args.points or w.N)
    if args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
