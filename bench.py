#!/usr/bin/env python
"""Benchmark of the SVD-Cache hot path on synthetic DiT-shaped feature streams.

One "step" is one caching interval of the schedule over every block of the stream: one
fused full step (project + residual + EMA, Eq. 8-11) followed by interval-1 fused cached
steps (forecast + reconstruct, Sec. 3.5), each as ONE batched launch over all blocks.
The metric is algorithmic HBM bytes per second over the whole step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload flux|hunyuan|dit_xl|tiny]
    python bench.py --impl reference      # the fp64 CPU oracle on the host cores

Under torchrun every rank runs its own copy of the stream (weak scaling, no data-path
collective); rank 0 prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2601_07396_b200 import streams  # noqa: E402

METRIC = "fused full/cached-step HBM GB/s and % of B200 HBM roofline (FLUX-shaped)"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0

# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of the timed kernels, from ncu
# captures of this very launch shape (all blocks of the workload in one batched launch; the
# summaries under profiles/ name the commands).  Keyed by (workload, blocks, kernel family);
# any other shape reports null -- nothing is scaled.
NCU_TRAFFIC_BYTES = {
    "cached": {("flux", 57, 2): 3269659648},   # profiles/umma_cached_kernel_flux_57blocks_traffic.txt
    "full": {("flux", 57, 2): 4303533312},     # profiles/umma_full_kernel_flux_57blocks_traffic.txt
}


def algorithmic_bytes(spec: streams.StreamSpec, nblocks: int):
    """Bytes the method must move per launch.  Full step: F in, R out, Chat read and written,
    its split-bf16 operand copy written (3 N k fp32-sized arrays), the basis once.  Cached
    step: R in, Fhat out, the operand copy of Chat in, the basis once."""
    N, D, k, b = spec.rows, spec.D, spec.k, spec.elem_bytes
    full = 2 * N * D * b + 3 * N * k * 4 + D * k * b
    cached = 2 * N * D * b + N * k * 4 + D * k * b
    return full * nblocks, cached * nblocks


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        inside = [r for (t, r) in self.rows if t0 <= t <= t1] or [r for (_, r) in self.rows[-3:]]
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in inside:
            p = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(p[0])); smax.append(float(p[1]))
            except Exception:
                continue
            for nm, val in zip(names, p[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def reduce_max(value: float, world: int, device) -> float:
    """Max over ranks of a per-rank number (the timed region's duration)."""
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_blocks(spec, rank: int, nblocks: int):
    """Blocks of the stream that rank `rank` owns: every rank gets `nblocks` blocks of its
    own (block ids rank * spec.blocks + 0 ..), so ranks never share a block and the step
    kernels need no collective (weak scaling)."""
    first = rank * spec.blocks
    return list(range(first, first + nblocks))


def whole_job_value(step_bytes: int, steps: int, world: int, max_ms: float) -> float:
    """GB/s of the whole job: bytes all ranks processed / the slowest rank's time."""
    return world * step_bytes * steps / (max_ms * 1e-3) / 1e9


# ------------------------------------------------------------------------- ours ---

def build_workload(spec, nblocks, device, block_offset=0, calibrate_rows=None):
    """Features, calibrated bases and reset states for `nblocks` blocks, resident on the
    device.  Returns dict of tensors."""
    from paper_2601_07396_b200 import binding as sc
    dt = sc.F32 if spec.dtype == "f32" else sc.BF16
    N, D, k = spec.rows, spec.D, spec.k
    F = torch.empty(nblocks, N, D, dtype=spec.torch_dtype, device=device)
    bases = torch.empty(nblocks, sc.svdcache_basis_bytes(D, k, dt), dtype=torch.uint8, device=device)
    ws = torch.empty(sc.svdcache_calibrate_workspace_bytes(D, k), dtype=torch.uint8, device=device)
    cal_ms = []
    n_cal = min(N, 4608) if calibrate_rows is None else calibrate_rows
    for b in range(nblocks):
        blk = block_offset + b
        st = streams.BlockStream(spec, blk, trajectory=0, device=device)
        st.features(0, out=F[b])
        if n_cal <= N:
            cal = streams.BlockStream(spec, blk, trajectory=1, device=device, rows=n_cal)
            stack = cal.features(0)
        else:   # several snapshots of the calibration trajectories, as many rows as asked for
            snaps = (n_cal + N - 1) // N
            per_traj = len(spec.calib_timesteps)
            stack = streams.calibration_stack(spec, blk, device=device,
                                              trajectories=tuple(range(1, 1 + (snaps + per_traj - 1) // per_traj)),
                                              timesteps=spec.calib_timesteps[:min(per_traj, snaps)])[:n_cal]
            cal = None
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        Vk, lam, tr, info = sc.svdcache_calibrate(stack, k, workspace=ws, strict=False)
        e1.record()
        torch.cuda.synchronize()
        cal_ms.append(e0.elapsed_time(e1))
        sc.svdcache_basis_prepare(Vk, dt, basis=bases[b])
        del st, cal, stack
    state = sc.new_state(N, D, k, dt, device, blocks=nblocks)
    Fhat = torch.empty_like(F)
    torch.cuda.synchronize()
    return dict(F=F, bases=bases, state=state, Fhat=Fhat, dt=dt, cal_ms=cal_ms, cal_rows=n_cal)


def measure_steps(sc, spec, wl, steps, warmup, barrier, sampler=None):
    """`warmup` untimed steps, then `steps` timed ones (one step = one batched full step + interval-1
    batched cached steps over all blocks of `wl`), CUDA events on the launching stream around the
    whole region and around every launch."""
    F, bases, state, Fhat = wl["F"], wl["bases"], wl["state"], wl["Fhat"]
    k, beta, interval = spec.k, spec.beta, spec.interval

    def one_step(events=None):
        if events is not None:
            e = torch.cuda.Event(enable_timing=True); e.record(); events.append(e)
        sc.svdcache_full_step_batched(F, bases, state, k, beta)
        if events is not None:
            e = torch.cuda.Event(enable_timing=True); e.record(); events.append(e)
        for j in range(1, interval):
            sc.svdcache_cached_step_batched(state, bases, Fhat, k, steps_since_full=j)
            if events is not None:
                e = torch.cuda.Event(enable_timing=True); e.record(); events.append(e)

    for _ in range(warmup):
        one_step()
    barrier()
    if sampler is not None:
        sampler.start()
        t_wait = time.time()
        while not sampler.rows and time.time() - t_wait < 3.0:   # nvidia-smi can take a second to print its first line
            time.sleep(0.02)
        time.sleep(0.05)
    launches0 = sc.svdcache_kernel_launches()
    events = []
    t_host0 = time.time()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(steps):
        one_step(events)
    stop.record()
    barrier()
    t_host1 = time.time()
    clocks = sampler.stop(t_host0, t_host1) if sampler is not None else None
    launches = sc.svdcache_kernel_launches() - launches0
    per = interval + 1
    full_ms, cached_ms = [], []
    for s_ in range(steps):
        ev = events[s_ * per:(s_ + 1) * per]
        full_ms.append(ev[0].elapsed_time(ev[1]))
        for j in range(1, interval):
            cached_ms.append(ev[j].elapsed_time(ev[j + 1]))
    return dict(total_ms=start.elapsed_time(stop), full_ms=full_ms, cached_ms=cached_ms, launches=launches, clocks=clocks)


def parity_of_timed_buffers(sc, spec, wl, rows_per_block=256):
    """Outside the timed region: the state and Fhat the timed launches left behind, sampled rows of
    the first, the middle and the last block, against the fp64 oracle driven through as many full
    steps (of the same F) as the state has seen.  Returns the worst relative Frobenius errors and
    raises SystemExit when a bound of the parity tests is exceeded."""
    from oracle import svdcache_oracle as oracle
    import numpy as np
    F, bases, state, Fhat, dt = wl["F"], wl["bases"], wl["state"], wl["Fhat"], wl["dt"]
    nb, N, D = F.shape
    k = spec.k
    beta = float(np.float32(spec.beta))
    rows = streams.sample_rows(N, rows_per_block, tile=128)
    rows_d = rows.to(F.device)
    worst = {"Chat": 0.0, "R": 0.0, "Fhat": 0.0}
    checked = sorted({0, nb // 2, nb - 1})
    steps_seen = 0
    for b in checked:
        steps_seen, status = sc.svdcache_state_query(state[b])
        if status != 0 or steps_seen < 1:
            raise SystemExit(f"bench parity: block {b} has status {status} after {steps_seen} full steps")
        V = (sc.basis_views(bases[b], D, k, dt)[0 if dt == sc.F32 else 2]).double().cpu().numpy()
        Fh = F[b][rows_d].double().cpu().numpy()
        chat = None
        for _ in range(int(steps_seen)):
            C, R, chat = oracle.full_step(Fh, V, beta, chat)
        ref = oracle.cached_step(chat, V, R)
        chat_v, r_v = sc.state_views(state[b], N, D, k, dt)
        for name, got, want in (("Chat", chat_v[rows_d], chat), ("R", r_v[rows_d], R), ("Fhat", Fhat[b][rows_d], ref)):
            g = got.double().cpu().numpy()
            err = float(np.linalg.norm(g - want) / np.linalg.norm(want))
            worst[name] = max(worst[name], err)
    io_bound = 1e-5 if dt == sc.F32 else 5e-3
    chat_bound = 1e-5 if dt == sc.F32 else max(1e-5, 4e-9 * D)
    bounds = {"Chat": chat_bound, "R": io_bound, "Fhat": io_bound}
    bad = {n_: e for n_, e in worst.items() if not e <= bounds[n_]}
    if bad:
        raise SystemExit(f"bench parity failed: {bad} against {bounds}")
    return {"rows": int(len(rows)) * len(checked), "blocks": checked, "full_steps_replayed": int(steps_seen),
            "Chat": worst["Chat"], "R": worst["R"], "Fhat": worst["Fhat"], "bounds": bounds,
            "against": "fp64 oracle on sampled rows of the buffers the timed launches wrote"}


def roofline_objects(spec, nblocks, full_ms, cached_ms, peak, peak_kind, path_used):
    b_full, b_cached = algorithmic_bytes(spec, nblocks)
    c_ms = sum(cached_ms) / max(1, len(cached_ms))
    f_ms = sum(full_ms) / max(1, len(full_ms))
    c_gbs = b_cached / (c_ms * 1e-3) / 1e9 if cached_ms else None
    f_gbs = b_full / (f_ms * 1e-3) / 1e9
    roof = {"bound": "hbm", "kernel": "cached step (batched)",
            "achieved": round(c_gbs, 2) if c_gbs else None, "peak": peak,
            "peak_source": f"{peak_kind} copy bandwidth", "unit": "GB/s",
            "frac": round(c_gbs / peak, 4) if c_gbs else None,
            "frac_of_nominal_8TBs": round(c_gbs / NOMINAL_HBM_GBS, 4) if c_gbs else None,
            "traffic": NCU_TRAFFIC_BYTES["cached"].get((spec.name, nblocks, path_used)),
            "algorithmic_bytes": b_cached, "avg_launch_ms": round(c_ms, 4)}
    roof_full = {"bound": "hbm", "kernel": "full step (batched)", "achieved": round(f_gbs, 2),
                 "peak": peak, "unit": "GB/s", "frac": round(f_gbs / peak, 4),
                 "frac_of_nominal_8TBs": round(f_gbs / NOMINAL_HBM_GBS, 4),
                 "traffic": NCU_TRAFFIC_BYTES["full"].get((spec.name, nblocks, path_used)),
                 "algorithmic_bytes": b_full, "avg_launch_ms": round(f_ms, 4)}
    return roof, roof_full


def hunyuan_addendum(sc, args, device, peak, peak_kind):
    """The same two kernels on the HunyuanVideo-shaped stream (N = 118,800 rows, k = 128): 8 of its
    60 blocks resident at a time (about 19 GB with state; every launch streams > 11 GB), fewer
    steps.  The headline value stays the FLUX-shaped one."""
    spec = streams.SPECS["hunyuan"]
    nblocks = 8
    wl = build_workload(spec, nblocks, device)
    steps = max(3, min(args.steps, 6))
    sampler = ClockSampler(device.index or 0)
    m = measure_steps(sc, spec, wl, steps, 3, torch.cuda.synchronize, sampler)
    path_used = sc.svdcache_last_path()
    roof, roof_full = roofline_objects(spec, nblocks, m["full_ms"], m["cached_ms"], peak, peak_kind, path_used)
    b_full, b_cached = algorithmic_bytes(spec, nblocks)
    step_bytes = b_full + (spec.interval - 1) * b_cached
    out = {"config": {"workload": "hunyuan-shaped stream", "blocks": nblocks, "rows": spec.rows, "D": spec.D,
                      "k": spec.k, "interval": spec.interval, "steps": steps, "warmup": 3},
           "value": round(step_bytes * steps / (m["total_ms"] * 1e-3) / 1e9, 2), "unit": "GB/s",
           "ms_per_step": round(m["total_ms"] / steps, 4),
           "roofline": roof, "roofline_full_step": roof_full,
           "tokens_blocks_per_s": round(spec.rows * nblocks * spec.interval * steps / (m["total_ms"] * 1e-3), 1),
           "gpu_launches": int(m["launches"]), "clocks": m["clocks"]}
    if not args.no_parity:
        out["parity"] = parity_of_timed_buffers(sc, spec, wl)
    return out


def run_ours(args):
    from paper_2601_07396_b200 import binding as sc
    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    sc.lib()

    spec = streams.SPECS[args.workload]
    nblocks = args.blocks or (spec.blocks if spec.name != "hunyuan" else 8)
    wl = build_workload(spec, nblocks, device, block_offset=rank_blocks(spec, rank, nblocks)[0],
                        calibrate_rows=args.calib_rows or None)
    F, bases, state, Fhat, dt = wl["F"], wl["bases"], wl["state"], wl["Fhat"], wl["dt"]
    k, beta, interval = spec.k, spec.beta, spec.interval
    bytes_full, bytes_cached = algorithmic_bytes(spec, nblocks)
    step_bytes = bytes_full + (interval - 1) * bytes_cached

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: K steps, CUDA events on the launching stream ----
    sampler = ClockSampler(local)
    m = measure_steps(sc, spec, wl, args.steps, args.warmup, barrier, sampler)
    clocks, launches = m["clocks"], m["launches"]
    total_ms = reduce_max(m["total_ms"], world, device)
    full_ms, cached_ms = m["full_ms"], m["cached_ms"]
    path_used = sc.svdcache_last_path()

    # ---- end to end: host buffers, H2D of F and D2H of the final Fhat every step ----
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    F_host = torch.empty(F.shape, dtype=F.dtype, pin_memory=True)
    F_host.copy_(F)
    out_host = torch.empty(Fhat.shape, dtype=Fhat.dtype, pin_memory=True)
    h2d = F_host.numel() * F_host.element_size()
    d2h = out_host.numel() * out_host.element_size()
    barrier()
    # The blocks are independent, so the step is pipelined over groups of blocks on a few streams:
    # while one group computes, the next one's F is on its way in and the previous one's Fhat on
    # its way out (PCIe is full duplex).  The result is that of one batched step over all blocks.
    ngroups = min(nblocks, 8)
    bounds = [(g * nblocks) // ngroups for g in range(ngroups + 1)]
    streams_ = [torch.cuda.Stream(device=device) for _ in range(min(3, ngroups))]
    main = torch.cuda.current_stream()
    s2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s2.record()
    for _ in range(e2e_steps):
        for st in streams_:
            st.wait_stream(main)
        for g in range(ngroups):
            b0, b1 = bounds[g], bounds[g + 1]
            st = streams_[g % len(streams_)]
            with torch.cuda.stream(st):
                F[b0:b1].copy_(F_host[b0:b1], non_blocking=True)
                sc.svdcache_full_step_batched(F[b0:b1], bases[b0:b1], state[b0:b1], k, beta, stream=st)
                for j in range(1, interval):
                    sc.svdcache_cached_step_batched(state[b0:b1], bases[b0:b1], Fhat[b0:b1], k, steps_since_full=j,
                                                    stream=st)
                out_host[b0:b1].copy_(Fhat[b0:b1], non_blocking=True)
        for st in streams_:
            main.wait_stream(st)
    e2.record()
    barrier()
    e2e_ms = reduce_max(s2.elapsed_time(e2), world, device)

    if rank != 0:
        return
    peak, peak_kind = measured_peak()
    value = whole_job_value(step_bytes, args.steps, world, total_ms)
    e2e_value = whole_job_value(step_bytes, e2e_steps, world, e2e_ms)
    roof, roof_full = roofline_objects(spec, nblocks, full_ms, cached_ms, peak, peak_kind, path_used)
    line = {
        "metric": METRIC, "value": round(value, 2), "unit": "GB/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(total_ms / args.steps, 4),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if spec.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": f"{spec.name}-shaped stream", "blocks": nblocks, "rows": spec.rows,
                   "D": spec.D, "k": spec.k, "interval": interval, "beta": beta,
                   "step": f"1 batched full step + {interval - 1} batched cached steps over all blocks",
                   "l2": "inputs larger than L2 (each launch streams >= 1 GB)" if step_bytes > 6e8 else
                         "inputs smaller than L2: launch-bound parity config, not a roofline config",
                   "kernel_family": {1: "cuda-core", 2: "tcgen05"}.get(path_used, "?"),
                   "library": sc.LIB_PATH,
                   "parallelism": f"blocks replicated per rank x{world}, no collective"},
        "roofline": roof,
        "roofline_full_step": roof_full,
        "tokens_blocks_per_s": round(world * spec.rows * nblocks * interval * args.steps / (total_ms * 1e-3), 1),
        "e2e": {"value": round(e2e_value, 2), "unit": "GB/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                "note": "pinned host F copied in and final Fhat copied out every step, pipelined over groups of blocks on 3 streams"},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "calibration": {"rows": wl["cal_rows"], "median_ms_per_block": round(statistics.median(wl["cal_ms"]), 3),
                        "note": "one-off per block, outside the timed steps"},
    }
    if not args.no_parity:
        line["parity"] = parity_of_timed_buffers(sc, spec, wl)
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(spec, F, bases, dt, budget_s=args.cpu_seconds)
    if world == 1 and spec.name == "flux" and not args.blocks and not args.no_hunyuan:
        del F, bases, state, Fhat, F_host, out_host, wl
        torch.cuda.empty_cache()
        line["hunyuan"] = hunyuan_addendum(sc, args, device, peak, peak_kind)
    print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# -------------------------------------------------------------- oracle-timed legs ---

def _oracle_interval(oracle, Fh, V, beta, interval):
    C, R, chat = oracle.full_step(Fh, V, beta, None)
    for _ in range(interval - 1):
        oracle.cached_step(chat, V, R)


def cpu_baseline(spec, F, bases, dt, budget_s=12.0):
    """The fp64 oracle as it stands, timed on this machine's host cores over whole blocks of
    the same workload until `budget_s` seconds have been spent."""
    from oracle import svdcache_oracle as oracle
    from paper_2601_07396_b200 import binding as sc
    import numpy as np
    nb = F.shape[0]
    rows = min(spec.rows, 2048)
    done_bytes, t_spent, used = 0, 0.0, 0
    sub = streams.StreamSpec(**{**spec.__dict__, "rows": rows})
    bf, bc = algorithmic_bytes(sub, 1)
    b = -1
    while t_spent < budget_s:
        b = (b + 1) % nb
        V = (sc.basis_views(bases[b], spec.D, spec.k, dt)[0 if dt == sc.F32 else 2]).double().cpu().numpy()
        Fh = F[b, :rows].double().cpu().numpy()
        t0 = time.perf_counter()
        _oracle_interval(oracle, Fh, V, float(np.float32(spec.beta)), spec.interval)
        t_spent += time.perf_counter() - t0
        done_bytes += bf + (spec.interval - 1) * bc
        used += 1
    return {"value": round(done_bytes / t_spent / 1e9, 4), "unit": "GB/s", "cores": oracle.threads(),
            "kind": "oracle",
            "sample": f"first {rows} rows of a block, {used} block passes: 1 full + {spec.interval - 1} cached steps each, "
                      f"{t_spent:.1f} s of CPU work"}


def run_reference(args):
    """Reference arm: the fp64 CPU oracle on the host cores, on a bounded sample of the
    same workload, metric and unit.  Rank 0 only."""
    rank, world, _ = dist_env()
    if rank != 0:
        return
    from oracle import svdcache_oracle as oracle
    import numpy as np
    spec = streams.SPECS[args.workload]
    rows = min(spec.rows, args.ref_rows)
    sub = streams.StreamSpec(**{**spec.__dict__, "rows": rows})
    st = streams.BlockStream(spec, 0, device="cpu", rows=rows)
    Fh = st.features(0).double().numpy()
    V = st.V_gen[:, :spec.k].to(spec.torch_dtype).double().numpy()
    bf, bc = algorithmic_bytes(sub, 1)
    step_bytes = bf + (spec.interval - 1) * bc
    beta = float(np.float32(spec.beta))
    for _ in range(args.warmup):
        _oracle_interval(oracle, Fh, V, beta, spec.interval)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        _oracle_interval(oracle, Fh, V, beta, spec.interval)
    dt_s = time.perf_counter() - t0
    value = step_bytes * args.steps / dt_s / 1e9
    sample = f"{rows} rows of block 0 of the {spec.name}-shaped stream per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": "GB/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(dt_s * 1e3 / args.steps, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{spec.name}-shaped stream", "rows": rows, "D": spec.D, "k": spec.k,
                   "interval": spec.interval, "sample": sample},
        "cpu_baseline": {"value": round(value, 4), "unit": "GB/s", "cores": oracle.threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": round(value, 4), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_sweep(args):
    """Rank and calibration sweep on the FLUX shape: one JSON line per rank k (both fused
    step kernels, batched over `--blocks` blocks) and per calibration stack size M (Gram on
    the tensor cores, then the eigen-solver).  One GPU; not the headline line."""
    from paper_2601_07396_b200 import binding as sc
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    device = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    peak, peak_kind = measured_peak()
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            tf_peak = float(json.load(fh)["bf16_tflops"])
    except Exception:
        tf_peak = 1590.0
    base = streams.FLUX
    nb = args.blocks or 16
    N, D = base.rows, base.D

    def timed(fn, reps):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    F = torch.empty(nb, N, D, dtype=torch.bfloat16, device=device)
    for b in range(nb):
        streams.BlockStream(base, b, device=device).features(0, out=F[b])
    Fhat = torch.empty_like(F)
    V_gen = streams.BlockStream(base, 0, device=device).V_gen     # D x 256, orthonormal
    for k in streams.SWEEP_RANKS:
        spec = streams.StreamSpec(**{**base.__dict__, "k": k})
        Vk = V_gen[:, :k].float().contiguous()
        bases = torch.empty(nb, sc.svdcache_basis_bytes(D, k, sc.BF16), dtype=torch.uint8, device=device)
        for b in range(nb):
            sc.svdcache_basis_prepare(Vk, sc.BF16, basis=bases[b])
        state = sc.new_state(N, D, k, sc.BF16, device, blocks=nb)
        bf, bc = algorithmic_bytes(spec, nb)
        ms_f = timed(lambda: sc.svdcache_full_step_batched(F, bases, state, k, spec.beta), args.steps)
        ms_c = timed(lambda: sc.svdcache_cached_step_batched(state, bases, Fhat, k), args.steps)
        gf, gc = bf / ms_f / 1e6, bc / ms_c / 1e6
        # split-bf16 operand: 2 N D k flops in pass 1, 4 N D k in pass 2 / the cached product
        tf_f, tf_c = nb * 6.0 * N * D * k / ms_f / 1e9, nb * 4.0 * N * D * k / ms_c / 1e9
        print(json.dumps({"sweep": "rank", "k": k, "blocks": nb, "rows": N, "D": D,
                          "full_step": {"ms": round(ms_f, 4), "GBps": round(gf, 1), "frac_hbm": round(gf / peak, 4),
                                        "TFLOPs": round(tf_f, 1), "frac_tensor": round(tf_f / tf_peak, 4)},
                          "cached_step": {"ms": round(ms_c, 4), "GBps": round(gc, 1), "frac_hbm": round(gc / peak, 4),
                                          "TFLOPs": round(tf_c, 1), "frac_tensor": round(tf_c / tf_peak, 4)},
                          "peaks": {"hbm_GBps": peak, "bf16_TFLOPs": tf_peak, "source": peak_kind}}), flush=True)
        del state, bases
    # ---- modes beyond the method's own step (Sec. 4.5, Sec. 5.3), at the FLUX rank: bytes and time per mode ----
    k = base.k
    Vk = V_gen[:, :k].float().contiguous()
    bases = torch.empty(nb, sc.svdcache_basis_bytes(D, k, sc.BF16), dtype=torch.uint8, device=device)
    for b in range(nb):
        sc.svdcache_basis_prepare(Vk, sc.BF16, basis=bases[b])
    state = sc.new_state(N, D, k, sc.BF16, device, blocks=nb)
    bf, bc = algorithmic_bytes(base, nb)
    hist = [torch.empty(nb, N, k, dtype=torch.float32, device=device) for _ in range(3)]
    for h in hist:
        sc.svdcache_full_step_batched(F, bases, state, k, base.beta, C_out=h)
    fbuf = torch.empty(nb, sc.svdcache_forecast_bytes(N, k), dtype=torch.uint8, device=device)
    modes = [
        ("full step, EMA on the principal part, residual reused (the method)", bf,
         lambda: sc.svdcache_full_step_batched(F, bases, state, k, base.beta)),
        ("full step, reuse on both (beta = 0)", bf,
         lambda: sc.svdcache_full_step_batched(F, bases, state, k, 0.0)),
        ("full step, EMA on both (beta_R = 0.5; reads the old R as well)", bf + nb * N * D * 2,
         lambda: sc.svdcache_full_step_residual_ema_batched(F, bases, state, k, base.beta, 0.5)),
        ("cached step, EMA forecast (the method)", bc,
         lambda: sc.svdcache_cached_step_batched(state, bases, Fhat, k)),
    ]
    for order in (1, 2):
        modes.append((f"cached step, Newton forecast of order {order} (history read, forecast written, 2 launches)",
                      bc + nb * N * k * 4 * (order + 1) + nb * N * k * 8,
                      lambda order=order: sc.svdcache_cached_step_forecast_batched(
                          state, bases, Fhat, k, hist[:order + 1], sc.PREDICT_NEWTON, 3, base.interval, forecast=fbuf)))
    for name, nbytes, fn in modes:
        ms = timed(fn, args.steps)
        print(json.dumps({"sweep": "mode", "mode": name, "k": k, "blocks": nb, "algorithmic_bytes": nbytes,
                          "ms": round(ms, 4), "GBps": round(nbytes / ms / 1e6, 1), "frac_hbm": round(nbytes / ms / 1e6 / peak, 4)}),
              flush=True)
    del state, bases, hist, fbuf
    del F, Fhat
    torch.cuda.empty_cache()
    k = base.k
    for M in streams.SWEEP_CALIB_ROWS:
        snaps = max(1, M // N)
        stack = streams.calibration_stack(base, 0, device=device,
                                          trajectories=tuple(range(1, 1 + (snaps + 7) // 8)),
                                          timesteps=base.calib_timesteps[:min(8, snaps)])[:M]
        ws = torch.empty(sc.svdcache_calibrate_workspace_bytes(D, k), dtype=torch.uint8, device=device)

        def gram():
            sc.svdcache_calibrate_begin(D, k, ws)
            sc.svdcache_calibrate_accumulate(stack, ws)
        ms_g = timed(gram, 3)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        Vk, lam, tr, info = sc.svdcache_calibrate_finish(D, k, ws, strict=False)
        e1.record()
        torch.cuda.synchronize()
        tf = 2.0 * M * D * D / ms_g / 1e9
        # the kernel computes the 128 x 256 tiles that touch the upper block triangle of G
        nbt = (D + 127) // 128
        tiles = sum(1 for i in range(nbt) for j in range((nbt + 1) // 2) if 2 * j + 1 >= i)
        issued = tf * tiles * 128 * 256 / float(D * D)
        print(json.dumps({"sweep": "calibration", "M": int(stack.shape[0]), "D": D, "k": k,
                          "gram": {"ms": round(ms_g, 3), "TFLOPs_full_square": round(tf, 1),
                                   "TFLOPs_issued": round(issued, 1), "frac_tensor": round(issued / tf_peak, 4),
                                   "note": "frac_tensor = MMA work issued (the tiles of the upper block triangle) over "
                                           "the measured bf16 GEMM peak; TFLOPs_full_square counts 2 M D^2"},
                          "eigen": {"ms": round(e0.elapsed_time(e1), 1), "multiplications_by_G": info[0],
                                    "max_rel_residual": info[1]}}), flush=True)
        del stack, ws


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20,
                    help="timed steps (20 FLUX steps are ~70 ms: short enough to stay under the power cap, like the "
                         "burst copy the roofline peak was measured with; several hundred steps run ~6 %% slower "
                         "at ~1.6 GHz with sw_power_cap active)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="flux", choices=sorted(streams.SPECS))
    ap.add_argument("--blocks", type=int, default=0, help="override the number of blocks")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--ref-rows", type=int, default=1024)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-parity", action="store_true", help="skip the oracle check of the timed buffers")
    ap.add_argument("--no-hunyuan", action="store_true", help="skip the HunyuanVideo-shaped addendum of the default run")
    ap.add_argument("--calib-rows", type=int, default=0, help="rows of the per-block calibration stack (default: min(N, 4608))")
    ap.add_argument("--sweep", action="store_true", help="rank and calibration sweep on the FLUX shape")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
