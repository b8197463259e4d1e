#!/usr/bin/env python
"""Benchmark of the suspend/resume hot path on B200.

One step = one pass of the whole path over one batch of synthetic suspended requests:
retain one request in HBM and resume it in place, suspend the batch to pinned host memory
(descriptor build, gather kernel, device-to-host copies, block release), expire one host
image and re-admit it, resume the batch (block allocation, host-to-device copies, scatter
kernel).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload llama3_8b|tiny|gqa64|trace|longctx|paper_70b_tp4|paper_shape]
                  [--route staged|mapped|dma2d] [--kernel warp|bulk] [--layout layer|block] [--arena host|device]
"""
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

from kvr_synth import CONFIGS, context_lengths, fill_bytes, free_order, occupancy_fillers  # noqa: E402

SEED = 20260830
METRIC = "suspend/resume payload GB/s (batched suspend to pinned host, then batched resume)"


def peaks():
    """Measured roofline denominators written by the driver, else the documented fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return json.load(open(path))["hbm_gbs"], "measured"
    return 6650.0, "fallback"


def l2_residues():
    """Bytes a mover launch has written but not yet evicted to DRAM when it ends (ncu capture on a small case:
    DRAM reads equal the payload, DRAM writes fall short of it by this constant), per kernel and direction; the
    summary under profiles/ carries them on one 'l2_residue_bytes' line."""
    path = os.path.join(ROOT, "profiles", "ncu_dram_traffic_movers.md")
    out = {}
    if os.path.exists(path):
        for line in open(path):
            if line.startswith("l2_residue_bytes "):
                for kv in line.split()[1:]:
                    k, v = kv.split("=")
                    out[k] = float(v)
    return out, "profiles/ncu_dram_traffic_movers.md"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        rows = [r for r in self.rows if len(r) == 6 and r[0].isdigit()]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[2 + i] == "Active" for r in rows)]
        return {"sm_mhz": float(np.median([int(r[0]) for r in rows])), "sm_max_mhz": float(rows[0][1]),
                "reasons": reasons, "samples": len(rows)}


def build_workload(name, n_requests_cap=None, overrides=None):
    """The named configuration; `overrides` (num_blocks, requests, fixed_tokens) shrink it for profiling."""
    import dataclasses
    w = CONFIGS[name]
    o = overrides or {}
    if o.get("num_blocks"):
        w = dataclasses.replace(w, num_blocks=o["num_blocks"])
    if o.get("requests"):
        w = dataclasses.replace(w, n_requests=o["requests"])
    if o.get("fixed_tokens"):
        w = dataclasses.replace(w, length_rule=("fixed", o["fixed_tokens"]))
    seed = SEED + list(CONFIGS).index(name)
    lens = context_lengths(w.length_rule, w.n_requests, seed)
    if n_requests_cap is not None:
        lens = lens[:n_requests_cap]
    bs = w.block_size
    used = int(sum(-(-int(n) // bs) for n in lens))
    fillers = occupancy_fillers(w.num_blocks, bs, used, w.occupancy, seed) if w.occupancy else np.zeros(0, np.int64)
    return w, seed, lens, fillers


def engine_kwargs(args, kvr):
    """Engine settings from the command line; 0 / unset leaves the library's own default in place."""
    kw = dict(chunk_bytes=args.chunk_mib << 20, staging_slots=args.slots, max_ctas=args.max_ctas,
              kernel={"warp": kvr.KERNEL_WARP, "bulk": kvr.KERNEL_BULK}[args.kernel],
              suspend_single_bytes=args.suspend_single_mib << 20, resume_single_bytes=args.resume_single_mib << 20,
              copy_piece_bytes=args.copy_piece_mib << 20)
    if args.bulk_shape:
        kw["bulk_shape"] = tuple(int(x) for x in args.bulk_shape.split(","))
    return kw


def staging_note(args):
    slot, n = (args.chunk_mib or 64), (args.slots or 32)
    return {"slot_mib": slot, "slots_per_direction": n, "staging_mib_total": 2 * slot * n,
            "largest_launch_mib": slot * (n - 1), "library_default": not (args.chunk_mib or args.slots)}


def cpu_oracle_sample(geom, tokens, threads=1):
    """Times the oracle's gather and scatter loops, as they stand, on one request of `tokens` tokens."""
    import oracle as orc
    L, H, D, e, BS = geom
    nb = -(-tokens // BS)
    NB = nb * 2
    pool = fill_bytes(SEED, 77, NB * BS * 2 * L * H * D * e, e).copy()
    rng = np.random.default_rng(SEED)
    src = rng.permutation(NB)[:nb].astype(np.int32)
    t0 = time.perf_counter()
    img = orc.gather(pool, L, H, D, e, BS, NB, src, tokens)
    t1 = time.perf_counter()
    dst = rng.permutation(NB)[:nb].astype(np.int32)
    orc.scatter(pool, img, L, H, D, e, BS, NB, dst, tokens)
    t2 = time.perf_counter()
    payload = img.size
    return {"payload_bytes": payload, "suspend_s": t1 - t0, "resume_s": t2 - t1,
            "gbs": 2 * payload / (t2 - t0) / 1e9}


def cpu_oracle_threads(geom, tokens, threads):
    """The same oracle loops, one request per thread (the C calls drop the GIL), over one shared host pool."""
    import oracle as orc
    L, H, D, e, BS = geom
    nb = -(-tokens // BS)
    NB = 2 * nb * threads
    pool = fill_bytes(SEED, 78, NB * BS * 2 * L * H * D * e, e).copy()
    perm = np.random.default_rng(SEED + 1).permutation(NB).astype(np.int32)
    src = [perm[i * nb:(i + 1) * nb] for i in range(threads)]
    dst = [perm[(threads + i) * nb:(threads + i + 1) * nb] for i in range(threads)]

    def work(i):
        img = orc.gather(pool, L, H, D, e, BS, NB, src[i], tokens)
        orc.scatter(pool, img, L, H, D, e, BS, NB, dst[i], tokens)
    ts = [threading.Thread(target=work, args=(i,)) for i in range(threads)]
    t0 = time.perf_counter()
    for t in ts:
        t.start()
    for t in ts:
        t.join()
    dt = time.perf_counter() - t0
    payload = threads * tokens * 2 * L * H * D * e
    return {"value": 2 * payload / dt / 1e9, "unit": "GB/s", "cores": threads, "seconds": dt,
            "sample": "%d requests of %d tokens, one oracle gather + scatter per thread" % (threads, tokens)}


def run_reference(args):
    """Reference arm: the CPU oracle, untuned, on the host cores; every step is a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w, seed, lens, fillers = build_workload(args.workload)
    tokens = 2048
    for _ in range(args.warmup):
        cpu_oracle_sample(w.geom, 256)
    times, gbs = [], []
    for _ in range(args.steps):
        r = cpu_oracle_sample(w.geom, tokens)
        times.append(r["suspend_s"] + r["resume_s"])
        gbs.append(r["gbs"])
    value = float(np.mean(gbs))
    sample = "one %d-token request of the %s geometry per step: oracle gather then scatter, 1 thread" % (tokens, w.name)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(times)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": w.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def copy_peak_same_run(torch, nbytes=2 << 30, reps=10):
    """torch's device-to-device copy on this very GPU, counted read + write like the driver's measured peak."""
    free_b, _ = torch.cuda.mem_get_info()
    if free_b < 2 * nbytes + (1 << 30):
        return None
    a = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    b = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    ts = []
    for _ in range(reps + 3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        b.copy_(a)
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    del a, b
    return 2 * nbytes / min(ts[3:]) / 1e6


def link_peak(torch, kvr_pool, arena_bytes, reps=10, payload=0):
    """Pinned-copy peak in each direction over the library's own arena (same placement), by the library's probe:
    a 2 GiB copy (the burst figure, the roofline's denominator) and, when a payload size is given, one contiguous
    copy of that size (what the host side sustains over tens of GiB; on some hosts it is several percent lower)."""
    n = min(arena_bytes // 4096 * 4096, 2 << 30)
    st, d2h, h2d = kvr_pool.probe_link(n, reps)
    if st != 0:
        raise SystemExit("kvr_probe_link failed with status %d" % st)
    out = {"bytes": n, "reps": reps, "how": "kvr_probe_link: cudaMemcpyAsync arena <-> device, best of reps",
           "d2h_best_gbs": d2h, "h2d_best_gbs": h2d}
    big = min(arena_bytes, payload, 32 << 30) // 4096 * 4096
    if big > 2 * n:
        st, d2h_s, h2d_s = kvr_pool.probe_link(big, 2)
        if st == 0:
            out.update({"sustained_bytes": big, "d2h_sustained_gbs": d2h_s, "h2d_sustained_gbs": h2d_s})
    return out


def run_longctx(args):
    """Long-context stress: half of the 128k-token requests are suspended while the other half resumes, on the
    library's two stream pairs, with and without a synthetic HBM-read load kernel running beside them."""
    import torch

    from paper_2608_30830_b200 import kvr
    from paper_2608_30830_b200.multi import env_ranks

    rank, world, local = env_ranks()
    if rank != 0:
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    w = CONFIGS["longctx"]
    seed = SEED + 4
    L, H, D, e, BS = w.geom
    bpt = kvr.bytes_per_token(L, H, D, e)
    n_tok = w.length_rule[1]
    n_req = args.requests or w.n_requests
    avail = int(open("/proc/meminfo").read().split("MemAvailable:")[1].split()[0]) * 1024
    free_dev, _ = torch.cuda.mem_get_info()
    load_bytes = 8 << 30
    while n_req > 2 and (n_req * n_tok * bpt + (16 << 30) > 0.75 * avail or
                         n_req * n_tok * bpt + load_bytes + (6 << 30) > free_dev):
        n_req -= 2
    NB = n_req * (n_tok // BS)
    host_cap = n_req * n_tok * bpt + (64 << 20)
    dev_pool = torch.empty(NB * BS * bpt, dtype=torch.uint8, device="cuda")
    gen = torch.Generator(device="cuda").manual_seed(seed)
    view = dev_pool.view(torch.bfloat16)
    for i in range(0, view.numel(), 1 << 28):
        view[i:i + (1 << 28)].normal_(generator=gen)
    load_buf = torch.empty(load_bytes, dtype=torch.uint8, device="cuda").fill_(3)
    sink = torch.zeros(1024, dtype=torch.int64, device="cuda")
    torch.cuda.synchronize()
    pool = kvr.Pool(*w.geom, NB, host_cap, initial_free_order=free_order(seed, NB), device=local,
                    device_pool=dev_pool.data_ptr(), flags=kvr.PROFILE, **engine_kwargs(args, kvr))
    link = link_peak(torch, pool, host_cap)            # while the arena is still empty
    ids = list(range(n_req))
    for rid in ids:
        assert pool.admit(rid, n_tok)[0] == kvr.OK
    on_host, in_hbm = ids[:n_req // 2], ids[n_req // 2:]
    assert pool.suspend_to_host(on_host, kvr.SYNC)[0] == kvr.OK            # phase A, untimed
    half_bytes = (n_req // 2) * n_tok * bpt
    load_stream = torch.cuda.Stream()

    def load_rate(launches):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(load_stream):
            e0.record()
            assert kvr.read_load(load_buf.data_ptr(), load_bytes, launches, sink.data_ptr(), load_stream.cuda_stream) == kvr.OK
            e1.record()
        return e0, e1, launches * load_bytes

    def exchange(overlap, load_launches):
        nonlocal on_host, in_hbm
        ev = load_rate(load_launches) if load_launches else None
        t0 = time.perf_counter()
        assert pool.suspend_to_host(in_hbm)[0] == kvr.OK
        t_s = time.perf_counter() - t0
        if not overlap:
            assert pool.wait() == kvr.OK
        t1 = time.perf_counter()
        assert pool.resume_from_host(on_host)[0] == kvr.OK
        t_r = time.perf_counter() - t1
        assert pool.wait() == kvr.OK, kvr.last_error()
        wall = time.perf_counter() - t0
        sus = max(pool.latency(r)[2] for r in in_hbm) / 1e3
        res = max(pool.latency(r)[2] for r in on_host) / 1e3
        out = {"suspend_gbs": half_bytes / sus / 1e9, "resume_gbs": half_bytes / res / 1e9,
               "both_directions_gbs": 2 * half_bytes / wall / 1e9, "wall_s": wall,
               "suspend_call_ms": 1e3 * t_s, "resume_call_ms": 1e3 * t_r}
        if ev:
            torch.cuda.synchronize()
            out["load_gbs"] = ev[2] / ev[0].elapsed_time(ev[1]) / 1e6
        on_host, in_hbm = in_hbm, on_host
        return out

    def median_of(runs):
        return {k: float(np.median([r[k] for r in runs])) for k in runs[0]}

    exchange(True, 0)                                                      # warm-up
    e0, e1, nb = load_rate(200)
    torch.cuda.synchronize()
    load_alone = nb / e0.elapsed_time(e1) / 1e6
    sampler = ClockSampler(local)
    sampler.start()
    reps = max(args.steps, 1)
    peak, peak_kind = peaks()
    keys = ("gather_launches", "scatter_launches", "gather_bytes", "scatter_bytes", "gather_ms", "scatter_ms",
            "gather_kernel_ms", "scatter_kernel_ms")

    def phase(fn):
        """Run one phase; returns its result and the movers' roofline fractions over exactly its launches."""
        a = pool.stats()
        out = fn()
        b = pool.stats()
        d = {k: b[k] - a[k] for k in keys}
        fr = {}
        for side in ("gather", "scatter"):
            fr[side] = {"frac": 2 * d[side + "_bytes"] / max(d[side + "_ms"], 1e-9) / 1e6 / peak,
                        "in_kernel_frac": 2 * d[side + "_bytes"] / max(d[side + "_kernel_ms"], 1e-9) / 1e6 / peak,
                        "launches": int(d[side + "_launches"]),
                        "avg_launch_mib": d[side + "_bytes"] / max(d[side + "_launches"], 1) / 2**20}
        return out, fr
    seq, fr_seq = phase(lambda: median_of([exchange(False, 0) for _ in range(reps)]))
    ovl, fr_ovl = phase(lambda: median_of([exchange(True, 0) for _ in range(reps)]))
    # size the load so that it runs for most of the overlapped exchange
    launches = max(50, int(0.8 * ovl["wall_s"] * load_alone * 1e9 / load_bytes))
    ovl_load, fr_load = phase(lambda: median_of([exchange(True, launches) for _ in range(reps)]))
    clocks = sampler.stop()
    st = pool.stats()
    out = {
        "metric": "suspend/resume payload GB/s, both directions overlapped beside a synthetic HBM-read load",
        "value": ovl_load["both_directions_gbs"], "unit": "GB/s", "n_gpus": 1, "steps": reps, "warmup": 1,
        "ms_per_step": 1e3 * ovl_load["wall_s"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u8", "data": "synthetic",
        "config": {"workload": "longctx", "geometry": dict(zip(("layers", "kv_heads", "head_dim", "dtype_bytes", "block_size"), w.geom)),
                   "requests_requested": w.n_requests, "requests_run": n_req, "tokens_per_request": n_tok,
                   "bytes_per_direction": half_bytes, "num_blocks": NB, "load_buffer_bytes": load_bytes,
                   "kernel": args.kernel, "staging": staging_note(args), "max_ctas": args.max_ctas},
        "interference": {
            "alone_one_direction_at_a_time": seq, "overlapped": ovl, "overlapped_with_load": ovl_load,
            "load_alone_gbs": load_alone, "load_alone_frac_of_hbm_peak": load_alone / peak,
            "suspend_loss_pct_overlap": 100 * (1 - ovl["suspend_gbs"] / seq["suspend_gbs"]),
            "resume_loss_pct_overlap": 100 * (1 - ovl["resume_gbs"] / seq["resume_gbs"]),
            "suspend_loss_pct_overlap_and_load": 100 * (1 - ovl_load["suspend_gbs"] / seq["suspend_gbs"]),
            "resume_loss_pct_overlap_and_load": 100 * (1 - ovl_load["resume_gbs"] / seq["resume_gbs"]),
            "load_loss_pct": 100 * (1 - ovl_load["load_gbs"] / load_alone)},
        "host_link": link, "clocks": clocks,
        "roofline": {"bound": "hbm", "peak": peak, "unit": "GB/s", "tile_bytes": BS * H * D * e,
                     "by_phase": {"one_direction_at_a_time": fr_seq, "both_directions": fr_ovl,
                                  "both_directions_beside_the_load": fr_load},
                     "gather_frac": 2 * st["gather_bytes"] / max(st["gather_ms"], 1e-9) / 1e6 / peak,
                     "scatter_frac": 2 * st["scatter_bytes"] / max(st["scatter_ms"], 1e-9) / 1e6 / peak,
                     "gather_launches": int(st["gather_launches"]), "scatter_launches": int(st["scatter_launches"]),
                     "mover_busy_us_per_gb": {"gather": 1e3 * st["gather_ms"] / max(st["gather_bytes"] / 1e9, 1e-9),
                                              "scatter": 1e3 * st["scatter_ms"] / max(st["scatter_bytes"] / 1e9, 1e-9)},
                     "note": "CUDA events around every mover launch, all phases of this run"},
        "gpu_launches": int(st["gather_launches"] + st["scatter_launches"]),
    }
    print(json.dumps(out))
    pool.close()


def run_trace(args):
    """Mixed tiering trace: 256 requests arrive, suspend at an approval gate and resume after a drawn wait; the live
    controller (grace period in HBM, offload, one-shot timers, replay admission) decides every move.  Events run back
    to back (time-compressed); the virtual clock only drives the policy."""
    import torch

    from kvr_synth import event_trace, wait_mixture
    from paper_2608_30830_b200 import kvr
    from paper_2608_30830_b200.multi import env_ranks

    rank, world, local = env_ranks()
    if rank != 0:
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    w = CONFIGS["trace"]
    seed = SEED + 3
    L, H, D, e, BS = w.geom
    bpt = kvr.bytes_per_token(L, H, D, e)
    lengths = context_lengths(w.length_rule, w.n_requests, seed)
    host_cap = 32 << 30
    dev_pool = torch.empty(w.num_blocks * BS * bpt, dtype=torch.uint8, device="cuda")
    view = dev_pool.view(torch.bfloat16)
    gen = torch.Generator(device="cuda").manual_seed(seed)
    for i in range(0, view.numel(), 1 << 28):
        view[i:i + (1 << 28)].normal_(generator=gen)
    torch.cuda.synchronize()
    pool = kvr.Pool(*w.geom, w.num_blocks, host_cap, initial_free_order=free_order(seed, w.num_blocks), device=local,
                    device_pool=dev_pool.data_ptr(), flags=kvr.PROFILE, **engine_kwargs(args, kvr))
    link = link_peak(torch, pool, host_cap)
    prices = (0.0176, 0.02, 1.91)                           # the paper's H100 NVL price vector, as context constants
    mean_img = float(np.mean(lengths)) * bpt
    w_ref = 0.5 * 1800.0 + 0.5 * 120.0 * float(np.exp(0.5))  # mean of this configuration's wait mixture
    lam = 2.0 * (host_cap / mean_img) / w_ref                # twice the critical load
    ctl = kvr.Controller(pool, prices, lam, w_ref, mean_image_bytes=mean_img, hbm_grace_s=60.0,
                         branch=kvr.BRANCH_TTL, admission=kvr.ADMIT_REPLAY)
    events, waits = event_trace(w.n_requests, seed, lam, 1e18, None)   # arrivals and resumes; the controller owns the timers
    sampler = ClockSampler(local)
    sampler.start()
    t0 = time.perf_counter()
    outcomes = {}
    for t, _, kind, rid in events:
        if kind == "arrive":
            st, _ = pool.admit(rid, int(lengths[rid]))
            if st != kvr.OK:
                raise SystemExit("trace: admission failed with status %d (pool too small for the retained set?)" % st)
            s = ctl.suspend(rid, t)
        elif kind == "resume":
            s = ctl.resume(rid, t)
            if s == kvr.RECOMPUTE:
                assert pool.admit(rid, int(lengths[rid]))[0] == kvr.OK     # the caller's re-prefill
            assert pool.release(rid) == kvr.OK
        else:
            continue
        outcomes[(kind, s)] = outcomes.get((kind, s), 0) + 1
    assert pool.wait() == kvr.OK, kvr.last_error()
    wall = time.perf_counter() - t0
    clocks = sampler.stop()
    st = pool.stats()
    cs = ctl.stats()
    moved = st["bytes_suspended"] + st["bytes_resumed"]
    peak, peak_kind = peaks()
    g_gbs = 2 * st["gather_bytes"] / max(st["gather_ms"], 1e-9) / 1e6
    s_gbs = 2 * st["scatter_bytes"] / max(st["scatter_ms"], 1e-9) / 1e6
    out = {
        "metric": "suspend/resume payload GB/s over a time-compressed tiering trace (host clock, every call included)",
        "value": moved / wall / 1e9, "unit": "GB/s", "n_gpus": 1, "steps": 1, "warmup": 0, "ms_per_step": 1e3 * wall,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": "trace", "requests": int(w.n_requests), "num_blocks": w.num_blocks, "host_capacity": host_cap,
                   "lambda_per_s": lam, "w_ref_s": w_ref, "hbm_grace_s": 60.0, "t2_s": cs["t2"], "branch": "cpu_ttl",
                   "admission": "replay", "kernel": args.kernel, "staging": staging_note(args)},
        "trace": {"bytes_suspended": st["bytes_suspended"], "bytes_resumed": st["bytes_resumed"],
                  "bytes_expired_from_host": st["bytes_expired_from_host"], "controller": cs,
                  "outcomes": {"%s:%d" % k: v for k, v in sorted(outcomes.items())},
                  "gpu_cost_per_request": cs["gpu_cost"] / w.n_requests},
        "roofline": {"bound": "hbm", "peak": peak, "unit": "GB/s", "gather_frac": g_gbs / peak, "scatter_frac": s_gbs / peak,
                     "gather_in_kernel_frac": 2 * st["gather_bytes"] / max(st["gather_kernel_ms"], 1e-9) / 1e6 / peak,
                     "scatter_in_kernel_frac": 2 * st["scatter_bytes"] / max(st["scatter_kernel_ms"], 1e-9) / 1e6 / peak,
                     "gather_launches": int(st["gather_launches"]), "scatter_launches": int(st["scatter_launches"]),
                     "mover_busy_us_per_gb": {"gather": 1e3 * st["gather_ms"] / max(st["gather_bytes"] / 1e9, 1e-9),
                                              "scatter": 1e3 * st["scatter_ms"] / max(st["scatter_bytes"] / 1e9, 1e-9)},
                     "note": "per-request moves of ~0.6 GiB, one launch each; *_frac is taken from CUDA events around every launch "
                             "(they include the tens of microseconds a completion takes while the copy engine is busy), "
                             "*_in_kernel_frac from the kernels' own first and last clock stamps"},
        "host_link": link, "clocks": clocks, "gpu_launches": int(st["gather_launches"] + st["scatter_launches"]),
    }
    print(json.dumps(out))
    ctl.close()
    pool.close()


def probe_links(group, pool, host_cap, payload, torch):
    """Every rank measures its own link over its own arena: once alone (ranks take turns between barriers) and once
    with all ranks copying at the same time, which shows what sharing the host's DRAM and root ports costs."""
    alone = None
    for r in range(group.world):
        group.barrier()
        if group.rank == r:
            alone = link_peak(torch, pool, host_cap, payload=payload if group.world == 1 else 0)
    group.barrier()
    together = None
    if group.world > 1:
        n = min(host_cap // 4096 * 4096, 2 << 30)
        st, d2h, h2d = pool.probe_link(n, 6)
        together = (d2h, h2d) if st == 0 else (0.0, 0.0)
        group.barrier()
    # everybody learns everybody's figures: a vector with this rank's slots filled, summed over ranks
    vec = [0.0] * (5 * group.world)
    vec[5 * group.rank:5 * group.rank + 5] = [alone["d2h_best_gbs"], alone["h2d_best_gbs"],
                                              together[0] if together else 0.0, together[1] if together else 0.0,
                                              float(pool.numa_node)]
    allv = group.sum(vec)
    per_rank = [{"rank": r, "d2h_alone_gbs": allv[5 * r], "h2d_alone_gbs": allv[5 * r + 1],
                 "d2h_all_ranks_at_once_gbs": allv[5 * r + 2] or None, "h2d_all_ranks_at_once_gbs": allv[5 * r + 3] or None,
                 "arena_numa_node": int(allv[5 * r + 4])} for r in range(group.world)]
    return alone, per_rank


def run_ours(args):
    import torch

    from paper_2608_30830_b200 import kvr
    from paper_2608_30830_b200.multi import Group, env_ranks, fit_requests

    rank, world, local = env_ranks()
    dry = args.dry_run
    if not dry:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
        torch.cuda.set_device(local)
    group = Group("gloo" if dry else "nccl", None if dry else torch.device("cuda", local))

    # every rank runs its own replica of the workload (own pool, own host link, own arena): weak scaling.
    # Scale rule: the arenas of all ranks come out of the same host DRAM; keep geometry and lengths and
    # reduce the request count when they would not fit in 60% of what is available.
    ov = {"num_blocks": args.num_blocks, "requests": args.requests, "fixed_tokens": args.fixed_tokens}
    w, seed, lens, fillers = build_workload(args.workload, None, ov)
    bpt = kvr.bytes_per_token(*w.geom[:4])
    L, H, D, e, BS = w.geom
    shared_blocks = 0 if args.no_share else int(w.extra.get("shared_tokens", 0)) // BS
    shared_tokens = shared_blocks * BS
    requested = len(lens)
    avail = int(open("/proc/meminfo").read().split("MemAvailable:")[1].split()[0]) * 1024
    keep = int(group.max([-fit_requests(lens - shared_tokens, bpt, avail, world)])[0]) * -1      # the same count on every rank
    if keep != requested:
        w, seed, lens, fillers = build_workload(args.workload, keep, ov)
    if shared_blocks:
        # the fillers were sized as if every request owned its prefix: recompute them for the shared layout
        used = shared_blocks + int(sum(-(-int(n) // BS) - shared_blocks for n in lens))
        fillers = occupancy_fillers(w.num_blocks, BS, used, w.occupancy, seed) if w.occupancy else fillers
    payload = int((lens - shared_tokens).sum()) * bpt
    lone_tokens = 8192
    small_k = int(np.argmin(fillers)) if len(fillers) else None     # request used for the retain / expire rows
    small_tokens = int(fillers[small_k]) if small_k is not None else 0
    unshared_extra = int(lens.sum()) * bpt if shared_blocks else 0   # the comparison pass without sharing needs room too
    host_cap = -(-(max(payload, unshared_extra) + len(lens) * 4096 + (lone_tokens + small_tokens) * bpt + (64 << 20)) // 4096) * 4096

    route = {"auto": kvr.ROUTE_AUTO, "staged": kvr.ROUTE_STAGED, "mapped": kvr.ROUTE_MAPPED, "dma2d": kvr.ROUTE_DMA2D}[args.route]
    layout = {"layer": kvr.LAYER_MAJOR, "block": kvr.BLOCK_MAJOR}[args.layout]
    dev_pool = dev_arena = None
    if dry:
        pool = kvr.Pool(*w.geom, w.num_blocks, host_cap, initial_free_order=free_order(seed, w.num_blocks),
                        flags=kvr.METADATA_ONLY, layout=layout)
    else:
        # pool bytes: bf16 N(0,1) drawn on the device from a seeded generator
        pool_bytes = w.num_blocks * BS * bpt
        dev_pool = torch.empty(pool_bytes, dtype=torch.uint8, device="cuda")
        gen = torch.Generator(device="cuda")
        gen.manual_seed(seed + rank)
        view = dev_pool.view(torch.bfloat16)
        step_elems = 1 << 28
        for i in range(0, view.numel(), step_elems):
            view[i:i + step_elems].normal_(generator=gen)
        torch.cuda.synchronize()
        dev_arena = None
        if args.arena == "device":
            dev_arena = torch.empty(host_cap, dtype=torch.uint8, device="cuda")
        elif args.arena == "peer":               # the next GPU's memory, reached over NVLink (needs a second GPU)
            if torch.cuda.device_count() < 2 or world > 1:
                raise SystemExit("--arena peer needs a second GPU and a single-rank run")
            dev_arena = torch.empty(host_cap, dtype=torch.uint8, device="cuda:%d" % ((local + 1) % torch.cuda.device_count()))
        pool = kvr.Pool(*w.geom, w.num_blocks, host_cap, initial_free_order=free_order(seed, w.num_blocks),
                        device=local, device_pool=dev_pool.data_ptr(), route=route,
                        host_arena=dev_arena.data_ptr() if dev_arena is not None else None,
                        flags=kvr.PROFILE, layout=layout, **engine_kwargs(args, kvr))

    # the link peaks, before anything lives in the arena: per rank, alone and all at once
    link, per_rank_links = (None, None)
    if not dry and dev_arena is None:
        link, per_rank_links = probe_links(group, pool, host_cap, payload, torch)

    # live set: the batch and the fillers, admitted in a seeded interleaved order (fragmented placement)
    ids = list(range(len(lens)))
    filler_ids = list(range(1000, 1000 + len(fillers)))
    PREFIX = 900
    if shared_blocks:
        assert pool.admit(PREFIX, shared_tokens)[0] == kvr.OK          # the system prefix, computed once
    order = [(i, int(n)) for i, n in zip(ids, lens)] + [(i, int(n)) for i, n in zip(filler_ids, fillers)]
    np.random.default_rng(seed).shuffle(order)
    for rid, n in order:
        if shared_blocks and rid < 900:
            st, _ = pool.admit_sharing(rid, n, PREFIX, shared_blocks)
        else:
            st, _ = pool.admit(rid, n)
        assert st == kvr.OK, (rid, n, st, kvr.last_error())
    if shared_blocks:
        assert pool.release(PREFIX) == kvr.OK                          # its blocks live on through the sharers' references
    occupancy = 1.0 - pool.stats()["blocks_free"] / w.num_blocks
    small = filler_ids[small_k] if small_k is not None else None

    def barrier():
        if not dry:
            torch.cuda.synchronize()
        group.barrier()

    last_resume_ms = []

    def one_step(batch=ids, low_latency=args.low_latency):
        """Returns (device_ms_suspend, device_ms_resume, wall_s)."""
        t0 = time.perf_counter()
        if small is not None:                          # HBM retention: nothing moves, resume is resident
            assert pool.retain_in_hbm([small])[0] == kvr.OK
            assert pool.resume_from_host([small])[0] == kvr.RESIDENT
        st, per = pool.suspend_to_host(batch)
        assert st == kvr.OK, (st, per, kvr.last_error())
        assert pool.wait() == kvr.OK, kvr.last_error()
        sus = 0.0 if dry else max(pool.latency(r)[2] for r in batch)
        if small is not None:                          # host copy expires, resume answers recompute, re-admit
            assert pool.suspend_to_host([small], kvr.SYNC)[0] == kvr.OK
            assert pool.expire([small])[0] == kvr.OK
            assert pool.resume_from_host([small])[0] == kvr.RECOMPUTE
            assert pool.admit(small, small_tokens)[0] == kvr.OK
        st, per = pool.resume_from_host(batch, kvr.LOW_LATENCY if low_latency else 0)
        assert st == kvr.OK, (st, per, kvr.last_error())
        assert pool.wait() == kvr.OK, kvr.last_error()
        per_req = [0.0 if dry else pool.latency(r)[2] for r in batch]
        last_resume_ms[:] = per_req
        res = max(per_req)
        return sus, res, time.perf_counter() - t0

    for _ in range(args.warmup):
        one_step()
    sampler = ClockSampler(local)
    s0 = pool.stats()
    barrier()
    if not dry:
        sampler.start()
    t_begin = time.perf_counter()
    steps = [one_step() for _ in range(args.steps)]
    barrier()
    wall = time.perf_counter() - t_begin
    clocks = sampler.stop() if not dry else None
    s1 = pool.stats()

    sus_ms = float(np.sum([s[0] for s in steps]))
    res_ms = float(np.sum([s[1] for s in steps]))
    dev_s = (sus_ms + res_ms) / 1e3
    dev_s, wall, sus_ms, res_ms = group.max([dev_s, wall, sus_ms, res_ms])    # the job is as slow as its slowest rank
    payload_all = group.sum([payload])[0]
    K = args.steps
    moved = 2.0 * payload_all * K                      # bytes suspended + bytes resumed, all ranks
    value = moved / dev_s / 1e9 if dev_s > 0 else None
    e2e = moved / wall / 1e9

    if rank == 0 and dry:
        d = {k: s1[k] - s0[k] for k in ("suspends", "resumes", "bytes_suspended", "bytes_resumed")}
        print(json.dumps({
            "metric": METRIC, "value": None, "unit": "GB/s", "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": 1e3 * wall / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "u8", "data": "synthetic", "dry_run": True,
            "config": {"workload": w.name, "requests_requested": requested, "requests_run": len(ids),
                       "note": "launcher and bookkeeping check without a GPU: metadata-only pools, gloo ranks, nothing moved"},
            "bookkeeping": {"bytes_suspended_per_step_all_ranks": payload_all,
                            "bytes_suspended_this_rank": int(d["bytes_suspended"]), "suspends_this_rank": int(d["suspends"])},
            "gpu_launches": 0}))

    if rank == 0 and not dry:
        # kernels inside the timed region (profiling events around every launch)
        d = {k: s1[k] - s0[k] for k in ("gather_launches", "scatter_launches", "gather_bytes", "scatter_bytes",
                                        "gather_ms", "scatter_ms", "gather_kernel_ms", "scatter_kernel_ms", "d2h_bytes", "h2d_bytes", "desc_bytes",
                                        "d2h_copies", "h2d_copies")}
        peak, peak_kind = peaks()
        g_gbs = 2 * d["gather_bytes"] / max(d["gather_ms"], 1e-9) / 1e6
        s_gbs = 2 * d["scatter_bytes"] / max(d["scatter_ms"], 1e-9) / 1e6
        slower = "gather" if g_gbs <= s_gbs else "scatter"
        name = "kvr::move_%s<%s>" % (args.kernel, slower)
        ach = min(g_gbs, s_gbs)
        # DRAM traffic per launch: ncu measured, for this kernel and direction on a small case, reads = payload and
        # writes = payload minus a constant residue still in L2 at kernel end; reads and writes grow with the payload
        residues, residue_file = l2_residues()
        launches = max(d[slower + "_launches"], 1)
        alg_per_launch = 2 * d[slower + "_bytes"] / launches
        residue = residues.get("%s_%s" % (slower, args.kernel))
        same_run = None if args.no_extras else copy_peak_same_run(torch)

        def side(gbs, key):
            n = max(d[key + "_launches"], 1)
            r = residues.get("%s_%s" % (key, args.kernel))
            alg = 2 * d[key + "_bytes"] / n
            return {"gbs": gbs, "frac": gbs / peak, "launches": d[key + "_launches"], "avg_us": 1e3 * d[key + "_ms"] / n,
                    "avg_launch_mib": d[key + "_bytes"] / n / 2**20, "algorithmic_bytes_per_launch": alg,
                    "traffic": None if r is None else max(alg - r, 0.0),
                    "mover_busy_us_per_gb": 1e3 * d[key + "_ms"] / max(d[key + "_bytes"] / 1e9, 1e-9)}
        roofline = {"bound": "hbm", "kernel": name, "achieved": ach, "peak": peak, "unit": "GB/s",
                    "copy_peak_this_gpu_this_run": same_run,
                    "frac": ach / peak, "peak_source": peak_kind + " copy bandwidth, read+write bytes",
                    "algorithmic_bytes_per_launch": alg_per_launch,
                    "traffic": None if residue is None else max(alg_per_launch - residue, 0.0),
                    "traffic_source": None if residue is None else
                    "%s: ncu dram__bytes_read.sum + dram__bytes_write.sum of this kernel and direction on a small case "
                    "(reads = payload, writes = payload - %.1f MB still in L2 at kernel end), applied to this run's "
                    "bytes per launch" % (residue_file, residue / 1e6),
                    "in_kernel": {
                        "what": "the same launches timed by the kernels themselves: earliest CTA start to latest CTA end "
                                "(%globaltimer), i.e. without the launch and completion latency the events include",
                        "gather_frac": 2 * d["gather_bytes"] / max(d["gather_kernel_ms"], 1e-9) / 1e6 / peak,
                        "scatter_frac": 2 * d["scatter_bytes"] / max(d["scatter_kernel_ms"], 1e-9) / 1e6 / peak},
                    "gather": side(g_gbs, "gather"), "scatter": side(s_gbs, "scatter")}

        # the kernels alone, at the size of the whole batch: HBM -> HBM
        alone = None
        free_b, _ = torch.cuda.mem_get_info()
        whole = int(lens.sum()) * bpt
        need = whole + len(ids) * 256
        if free_b > need + (2 << 30) and not args.no_extras:
            buf = torch.empty(need, dtype=torch.uint8, device="cuda")
            best = {}
            for direction, fn in (("gather", pool.export_to_device), ("scatter", pool.import_from_device)):
                ts = []
                for _ in range(5):
                    st, _ = fn(ids, buf.data_ptr(), need, kvr.SYNC)
                    assert st == kvr.OK, kvr.last_error()
                    ts.append(max(pool.latency(r)[2] for r in ids))
                best[direction] = {"best_gbs": 2 * whole / min(ts[2:]) / 1e6,
                                   "median_gbs": 2 * whole / float(np.median(ts[2:])) / 1e6}
                best[direction]["frac"] = best[direction]["median_gbs"] / peak
            alone = best
            del buf

        # resume latency of a lone 8192-token request
        lone = None
        if not args.no_extras and pool.admit(5000, lone_tokens)[0] == kvr.OK:
            sus_l, res_l, res_host = [], [], []
            for _ in range(5):
                t0 = time.perf_counter()
                assert pool.suspend_to_host([5000], kvr.SYNC)[0] == kvr.OK
                sus_l.append((time.perf_counter() - t0) * 1e3)
                t0 = time.perf_counter()
                assert pool.resume_from_host([5000], kvr.SYNC)[0] == kvr.OK
                res_l.append((time.perf_counter() - t0) * 1e3)
                res_host.append(pool.latency(5000)[1])
            lone = {"tokens": lone_tokens, "bytes": lone_tokens * bpt,
                    "suspend_ms_median": float(np.median(sus_l)), "resume_ms_median": float(np.median(res_l)),
                    "resume_enqueue_ms_median": float(np.median(res_host)),
                    "resume_gbs": lone_tokens * bpt / float(np.median(res_l)) / 1e6,
                    "timing": "host clock, call entry to return of the synchronous call"}
            pool.release(5000)

        # shared prefix: what the same contexts cost when every request owns its whole context
        sharing = None
        if shared_blocks:
            one = ids[0]
            t0 = time.perf_counter()
            assert pool.suspend_to_host([one], kvr.SYNC)[0] == kvr.OK
            t1 = time.perf_counter()
            assert pool.resume_from_host([one], kvr.SYNC)[0] == kvr.OK
            t2 = time.perf_counter()
            sharing = {"shared_tokens": shared_tokens, "context_tokens": int(lens[0]), "private_tokens": int(lens[0]) - shared_tokens,
                       "bytes_per_suspend": (int(lens[0]) - shared_tokens) * bpt,
                       "lone_suspend_ms": 1e3 * (t1 - t0), "lone_resume_ms": 1e3 * (t2 - t1),
                       "batch_suspend_ms": sus_ms / K, "batch_resume_ms": res_ms / K}
            if not args.no_extras:
                for rid in ids:
                    assert pool.release(rid) == kvr.OK
                ok = all(pool.admit(rid, int(n))[0] == kvr.OK for rid, n in zip(ids, lens))
                if ok:
                    u = [one_step(ids, False) for _ in range(2)][-1]
                    t0 = time.perf_counter()
                    assert pool.suspend_to_host([one], kvr.SYNC)[0] == kvr.OK
                    t1 = time.perf_counter()
                    assert pool.resume_from_host([one], kvr.SYNC)[0] == kvr.OK
                    t2 = time.perf_counter()
                    sharing["without_sharing"] = {"bytes_per_suspend": int(lens[0]) * bpt, "lone_suspend_ms": 1e3 * (t1 - t0),
                                                  "lone_resume_ms": 1e3 * (t2 - t1), "batch_suspend_ms": u[0], "batch_resume_ms": u[1]}
                    sharing["bytes_ratio"] = int(lens[0]) / (int(lens[0]) - shared_tokens)
                    sharing["lone_resume_speedup"] = sharing["without_sharing"]["lone_resume_ms"] / sharing["lone_resume_ms"]

        sus_gbs = payload_all * K / sus_ms / 1e6
        res_gbs = payload_all * K / res_ms / 1e6
        if link is None:        # device-memory tier: no host link on the path; the bound is HBM
            host_link = {"arena": "device memory", "suspend_gbs": sus_gbs, "resume_gbs": res_gbs,
                         "suspend_frac_of_hbm_peak": 2 * sus_gbs / world / peak, "resume_frac_of_hbm_peak": 2 * res_gbs / world / peak}
            if args.arena == "peer":             # bound by NVLink: 770 GB/s per direction measured for a peer copy on this machine
                host_link = {"arena": "peer GPU memory over NVLink", "suspend_gbs": sus_gbs, "resume_gbs": res_gbs,
                             "suspend_frac_of_peer_copy_770": sus_gbs / 770.0, "resume_frac_of_peer_copy_770": res_gbs / 770.0}
        else:
            host_link = dict(link)
            d2h_sum = sum(r["d2h_alone_gbs"] for r in per_rank_links)
            h2d_sum = sum(r["h2d_alone_gbs"] for r in per_rank_links)
            host_link.update({"suspend_gbs": sus_gbs, "suspend_frac_of_d2h_peak": sus_gbs / d2h_sum,
                              "resume_gbs": res_gbs, "resume_frac_of_h2d_peak": res_gbs / h2d_sum,
                              "per_rank": per_rank_links,
                              "peak_note": "fractions are against the sum over ranks of each rank's own link measured alone"})
            if "d2h_sustained_gbs" in link:
                host_link.update({"suspend_frac_of_d2h_sustained": sus_gbs / world / link["d2h_sustained_gbs"],
                                  "resume_frac_of_h2d_sustained": res_gbs / world / link["h2d_sustained_gbs"]})
        cpu = cpu_oracle_sample(w.geom, 256 if args.no_extras else 4096)
        sample = ("one %d-token request of this geometry (%.2f GiB payload): oracle gather then scatter, 1 thread"
                  % (256 if args.no_extras else 4096, cpu["payload_bytes"] / 2**30))
        out = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": 1e3 * wall / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "u8", "data": "synthetic",
            "config": {"workload": w.name, "geometry": dict(zip(("layers", "kv_heads", "head_dim", "dtype_bytes", "block_size"), w.geom)),
                       "num_blocks": w.num_blocks, "requests_requested": requested, "requests_run": len(ids),
                       "tokens": int(lens.sum()), "shared_prefix_tokens": shared_tokens, "payload_bytes_per_direction": payload,
                       "occupancy_before_suspend": occupancy, "route": args.route, "arena": args.arena, "layout": args.layout, "kernel": args.kernel,
                       "staging": staging_note(args), "low_latency_resume": bool(args.low_latency), "seed": seed,
                       "arena_numa_node": pool.numa_node,
                       "l2": "inputs (tens of GiB) are far larger than L2; no flush needed",
                       "timing": "value: CUDA events, first enqueued work to last byte landed, summed over the two batched moves of each step; e2e: host clock around the K steps"},
            "e2e": {"value": e2e, "unit": "GB/s",
                    "h2d_bytes_per_step": int((d["h2d_bytes"] + d["desc_bytes"]) / K),
                    "d2h_bytes_per_step": int(d["d2h_bytes"] / K)},
            "gpu_launches": int(d["gather_launches"] + d["scatter_launches"]),
            "clocks": clocks, "roofline": roofline, "kernels_alone": alone, "host_link": host_link,
            "resume_latency_8k": lone, "sharing": sharing,
            "resume_latency_in_batch": {
                "what": "device time from the batched resume's first enqueued work until each request's last byte landed "
                        "(requests complete in the order given); last timed step",
                "first_ms": float(min(last_resume_ms)), "median_ms": float(np.median(last_resume_ms)),
                "last_ms": float(max(last_resume_ms)),
                "batch_ms_per_8k_tokens": float(max(last_resume_ms)) * 8192.0 / float((lens - shared_tokens).sum())},
            "cpu_baseline": {"value": cpu["gbs"], "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample,
                             "suspend_s": cpu["suspend_s"], "resume_s": cpu["resume_s"],
                             "all_cores": None if args.no_extras else
                             cpu_oracle_threads(w.geom, 1024, min(os.cpu_count() or 1, 32))},
        }
        print(json.dumps(out))
    pool.close()
    group.close()


def run_alone_by_size(args):
    """The movers alone, launch size by launch size, beside the driver's plain device-to-device copy of the same
    bytes (what the HBM peak is measured with).  One request with a shuffled block table is exported to / imported
    from a device buffer (one launch each, no link involved); L2 is flushed before every launch; CUDA events; median
    of 10 after 2 warm-ups.  Prints one JSON line (not the bench contract's)."""
    import torch

    from paper_2608_30830_b200 import kvr

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(0)
    w = CONFIGS[args.workload]
    L, H, D, e, BS = w.geom
    bpt = kvr.bytes_per_token(L, H, D, e)
    nb = (32 << 30) // (BS * bpt)                                         # 32 GiB pool
    largest = 4 << 30
    kernel = {"warp": kvr.KERNEL_WARP, "bulk": kvr.KERNEL_BULK}[args.kernel]
    shape = tuple(int(x) for x in args.bulk_shape.split(",")) if args.bulk_shape else None
    pool = kvr.Pool(L, H, D, e, BS, nb, 64 << 20, initial_free_order=free_order(SEED, nb), chunk_bytes=1 << 20,
                    staging_slots=2, kernel=kernel, bulk_shape=shape)
    dst = torch.empty(largest, dtype=torch.uint8, device="cuda")
    src = torch.empty(largest, dtype=torch.uint8, device="cuda")
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    peak, peak_kind = peaks()
    rows = []
    for mib in (16, 64, 256, 1024, 2048, 4096):
        nbytes = (mib << 20) // (BS * bpt) * (BS * bpt)
        assert pool.admit(1, nbytes // bpt)[0] == kvr.OK
        ms = {"gather": [], "scatter": [], "copy": []}
        for it in range(12):
            for side, fn in (("gather", pool.export_to_device), ("scatter", pool.import_from_device)):
                flush.fill_(it)
                torch.cuda.synchronize()
                st, _ = fn([1], dst.data_ptr(), nbytes)
                assert st == kvr.OK and pool.wait() == kvr.OK, kvr.last_error()
                ms[side].append(pool.latency(1)[2])
            flush.fill_(it)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            dst[:nbytes].copy_(src[:nbytes])
            e1.record()
            torch.cuda.synchronize()
            ms["copy"].append(e0.elapsed_time(e1))
        gbs = {k: 2 * nbytes / float(np.median(v[2:])) / 1e6 for k, v in ms.items()}
        rows.append({"launch_mib": nbytes / 2**20, "gather_gbs": gbs["gather"], "scatter_gbs": gbs["scatter"],
                     "plain_copy_gbs": gbs["copy"], "gather_vs_copy": gbs["gather"] / gbs["copy"],
                     "scatter_vs_copy": gbs["scatter"] / gbs["copy"], "gather_frac_of_peak": gbs["gather"] / peak,
                     "scatter_frac_of_peak": gbs["scatter"] / peak})
        assert pool.release(1) == kvr.OK
    print(json.dumps({"what": "movers alone by launch size against torch copy_ of the same bytes (GB/s of read + written bytes)",
                      "workload_geometry": args.workload, "kernel": args.kernel, "peak": peak, "peak_kind": peak_kind, "rows": rows}))
    pool.close()


def relaunch_under_torchrun(args):
    """`python bench.py --gpus N` started plainly: start the N ranks (one per GPU) and pass their output through."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")               # the rank count must stay visible in the job's log
    return subprocess.call(cmd, env=env)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama3_8b", choices=list(CONFIGS))
    ap.add_argument("--route", default="staged", choices=["auto", "staged", "mapped", "dma2d"])
    ap.add_argument("--layout", default="layer", choices=["layer", "block"], help="pool layout: layer-major or block-major")
    ap.add_argument("--kernel", default="bulk", choices=["warp", "bulk"])
    ap.add_argument("--chunk-mib", type=int, default=0, help="staging slot size (0 = the library's default, 64)")
    ap.add_argument("--slots", type=int, default=0, help="staging slots per direction (0 = the library's default, 32)")
    ap.add_argument("--suspend-single-mib", type=int, default=0, help="largest suspend that goes in one launch (0 = library default, 1024)")
    ap.add_argument("--resume-single-mib", type=int, default=0, help="largest resume that goes in one launch (0 = library default, 256)")
    ap.add_argument("--copy-piece-mib", type=int, default=int(os.environ.get("KVR_COPY_PIECE_MIB", "0")),
                    help="largest single link copy (0 = library default, 64)")
    ap.add_argument("--bulk-shape", default=os.environ.get("KVR_BULK_SHAPE", ""), help="bulk mover shape: warps,stages,piece_bytes")
    ap.add_argument("--arena", default="host", choices=["host", "device", "peer"],
                    help="where the second tier lives: pinned host memory, this GPU's memory (stand-in for a peer), or the next GPU's")
    ap.add_argument("--max-ctas", type=int, default=0, help="cap on the movers' grid (0 = fill the GPU)")
    ap.add_argument("--num-blocks", type=int, default=0, help="shrink the pool (profiling captures)")
    ap.add_argument("--requests", type=int, default=0, help="override the request count")
    ap.add_argument("--fixed-tokens", type=int, default=0, help="give every request this many tokens")
    ap.add_argument("--low-latency", action="store_true", help="batched resume with KVR_LOW_LATENCY")
    ap.add_argument("--no-share", action="store_true", help="paper_shape: every request owns its whole context")
    ap.add_argument("--no-extras", action="store_true", help="skip kernels-alone, lone-request and CPU legs")
    ap.add_argument("--alone-by-size", action="store_true",
                    help="the movers alone, 16 MiB to 4 GiB per launch, beside a plain device copy (its own JSON line)")
    ap.add_argument("--dry-run", action="store_true",
                    help="launcher and bookkeeping check without a GPU: metadata-only pools, gloo ranks; moves nothing")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(relaunch_under_torchrun(args))
    if args.impl == "reference":
        run_reference(args)
    elif args.alone_by_size:
        run_alone_by_size(args)
    elif args.workload == "longctx":
        run_longctx(args)
    elif args.workload == "trace":
        run_trace(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
