#!/usr/bin/env python
"""Benchmark of the CCD compression cycle (one JSON line on stdout).

A step is one pass of the whole hot path over one batch of synthetic input:
append a chunk of new K/V rows behind the survivors, then one
``ipot_score_and_compress`` (NuC ranking, CaP scoring, per-head selection, in-place
K/V compaction) over all layers x streams x kv-heads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3|cfg2|cfg4|cfg5]
    python bench.py --impl reference ...      # the CPU checker, as it stands, on the host cores

With N > 1 (under torchrun) every rank runs an independent replica on its own GPU:
the cycle has no exchange step, so there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2410_01518_b200 import inputs  # noqa: E402

WORKLOADS = {"cfg2": 2, "cfg3": 3, "cfg4": 4, "cfg5": 5}
# the token-novelty producer alone (Eq. 3): (vocabulary, new tokens per step), bf16 logits, one stream
REFERENCE_BUDGET_S = 150.0   # wall-clock budget of a whole --impl reference run (the checker is slow by design)
NOVELTY_WORKLOADS = {"nuc32k": (32000, 2048), "nuc128k": (128256, 2048)}
# generation over a full pot alone: one new token's attention over all layers' units, configs[cfg - 1] shape
DECODE_WORKLOADS = {"decode3": 3, "decode4": 4, "decode5": 5}
SCORERS = {"auto": 0, "simt": 1, "tensor": 2, "warp_mma": 3, "sweeps": 4}
SCORER_KERNELS = {1: "cap_row_stats + cap_column_sums (fp32 FMA)", 2: "cap_score_tc_kernel (tcgen05, one sweep)",
                  3: "cap_row_stats_mma + cap_column_sums_mma (mma.sync)", 4: "cap_score_ts_kernel (tcgen05, two sweeps)"}
MIN_SAMPLED_S = 1.0   # the clock sampler should see at least this much of timed running
RING = 4  # distinct chunks / query sets cycled through
PREHEAT_S = 0.5  # untimed running before the warm-up steps, see main()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1400.0, "source": "fallback"}


def recorded_traffic(kernel: str, shape: str, units: int):
    """dram__bytes_read + dram__bytes_write of one launch, scaled to `units` from the capture on record."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    for row in open(path):
        f = row.split()
        if len(f) >= 4 and not row.startswith("#") and f[0] == kernel and f[1] == shape:
            return float(f[3]) * units / float(f[2])
    return None


def workload_shape(cfg):
    """(rows appended per step, rows in the pot when the cycle runs)."""
    n_new = cfg.pot_size - cfg.keep
    return n_new, cfg.pot_size


def gen_ring(cfg, n_new, cap_keys=False):
    """RING chunks of new K/V rows, CaP queries and novelty scores (numpy, storage dtype);
    with cap_keys also the CaP's own key rows (CaP-inclusive scoring)."""
    ring = []
    for i in range(RING):
        K, V = inputs.make_kv(cfg, n_new, chunk=1 + i)
        ring.append({"K": K, "V": V, "Q": inputs.make_q(cfg, 1 + i), "aux": inputs.make_aux(cfg, 1 + i)})
        if cap_keys:
            ring[-1]["K_cap"] = inputs.make_kcap(cfg, 1 + i)
    K0, V0 = inputs.make_kv(cfg, cfg.keep, chunk=0)
    return ring, K0, V0


class ClockSampler:
    """nvidia-smi clock / throttle samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        rows = [r.split(",") for r in open(self.f.name).read().strip().splitlines() if r.count(",") >= 8]
        os.unlink(self.f.name)
        sm, reasons = [], set()
        for r in rows:
            r = [x.strip() for x in r]
            try:
                sm.append(float(r[1]))
                out["sm_max_mhz"] = float(r[2])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out["sm_mhz"] = float(np.median(sm))
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


_CPU_KV = {}


def cpu_baseline(cfg, ring, K0, V0, n_units_sample, threads=None, rope=False, cap_rows_sample=None):
    """The checker, as it stands, on a sample of the units of one cycle (and, for a yet smaller sample, on the
    first `cap_rows_sample` CaP rows of every query head: its cost is proportional to the rows)."""
    import oracle
    if threads:
        oracle.set_threads(threads)
    t = ring[0]
    if cap_rows_sample:
        t = dict(t)
        t["Q"] = np.ascontiguousarray(t["Q"][:, :, :, :cap_rows_sample])
        if t.get("K_cap") is not None:
            t["K_cap"] = np.ascontiguousarray(t["K_cap"][:, :, :, :cap_rows_sample])
    key = (id(K0), id(ring))
    if _CPU_KV.get("key") != key:  # the pot of the sampled cycle is assembled once per run, outside every timed call
        _CPU_KV.update(key=key, K=np.concatenate([K0, ring[0]["K"]], axis=3), V=np.concatenate([V0, ring[0]["V"]], axis=3), loaded=False)
    K, V = _CPU_KV["K"], _CPU_KV["V"]
    units = np.linspace(0, cfg.units - 1, n_units_sample).astype(np.int32)
    rope = inputs.make_rope_table(cfg.pot_size, cfg.d, cfg.dtype) + (False,) if rope else None
    if not _CPU_KV["loaded"]:  # load the library
        oracle.cycle(t["Q"], K, V, t["aux"], cfg.keep, cfg.nuc_slots, units=units[:1], K_cap=t.get("K_cap"), rope=rope)
        _CPU_KV["loaded"] = True
    t0 = time.perf_counter()
    oracle.cycle(t["Q"], K, V, t["aux"], cfg.keep, cfg.nuc_slots, units=units, K_cap=t.get("K_cap"), rope=rope)
    dt = time.perf_counter() - t0
    cycles_per_s = (len(units) / cfg.units) / dt
    return cycles_per_s, dt, len(units), oracle.max_threads()


def whole_job_rate(ms_local: float, steps: int, world: int, device="cpu"):
    """Replicas-only aggregation: every rank ran `steps` independent cycles; the job's time is the
    slowest rank's.  Returns (cycles/s over all ranks, ms per step)."""
    ms = ms_local
    if world > 1:
        import torch
        import torch.distributed as dist
        t = torch.tensor([ms_local], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return world * steps * 1e3 / ms, ms / steps


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_new, N = workload_shape(cfg)
    small = cfg.with_layers(min(cfg.layers, 2))  # the sample only needs a few layers' tensors
    ring, K0, V0 = gen_ring(small, n_new, args.cap_keys)
    # every step is a bounded sample of the cycle, sized so that steps + warmup fit REFERENCE_BUDGET_S: 16 units with
    # all CaP rows while that fits, else one unit with as many of its CaP rows as the per-step share allows
    cpu_baseline(small, ring, K0, V0, 1, rope=args.rope)   # assembles the pot, loads the library
    t0 = time.perf_counter()
    cpu_baseline(small, ring, K0, V0, 1, rope=args.rope)
    t_unit = time.perf_counter() - t0                        # one unit, all CaP rows, with the call's overhead
    share = REFERENCE_BUDGET_S / max(1, args.steps + args.warmup)
    n_sample, p_sample = min(small.units, 16), cfg.cap_rows
    if share < 2.0 * t_unit:
        n_sample = 1
        p_sample = max(1, min(cfg.cap_rows, int(cfg.cap_rows * share / t_unit)))
    rows = None if p_sample == cfg.cap_rows else p_sample
    for _ in range(args.warmup):
        cpu_baseline(small, ring, K0, V0, 1, rope=args.rope, cap_rows_sample=rows)
    times = []
    for _ in range(args.steps):
        _, dt, n_units, threads = cpu_baseline(small, ring, K0, V0, n_sample, rope=args.rope, cap_rows_sample=rows)
        times.append(dt)
    ms = float(np.mean(times)) * 1e3 * (cfg.units / n_sample) * (cfg.cap_rows / p_sample)  # one full cycle, extrapolated
    value = 1e3 / ms
    line = {
        "impl": "reference", "metric": "ccd_cycles_per_s", "value": value, "unit": "cycles/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(cfg, n_new, N, args.cap_keys, getattr(args, "rope", False)),
        "cpu_baseline": {"value": value, "unit": "cycles/s", "cores": min(threads, n_sample), "kind": "oracle",
                         "sample": f"{n_sample} of {cfg.units} units, {p_sample} of {cfg.cap_rows} CaP rows per query head, of one "
                                   f"cycle per step (units are independent and equal-sized, the cost is proportional to "
                                   f"the rows); full-cycle time extrapolated"},
        "e2e": {"value": value, "unit": "cycles/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "pot_tokens_per_s": value * N * cfg.batch,
    }
    print(json.dumps(line))


def run_decode(args):
    """Generation over the pot alone: a step is one ipot_decode_attention call over every unit of a full pot."""
    cfg = inputs.CONFIGS[DECODE_WORKLOADS[args.workload]]
    if args.layers > 0:
        cfg = cfg.with_layers(args.layers)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    N = cfg.pot_size
    workload = (f"configs[{cfg.cfg_id - 1}] {cfg.name}: one new token attends to the full pot "
                f"({cfg.units} units x {N} rows)")
    rng = np.random.default_rng(cfg.seed)
    qs = [inputs.store(rng.standard_normal((cfg.layers, cfg.batch, cfg.Hq, cfg.d), dtype=np.float32), cfg.dtype) for _ in range(RING)]
    if args.impl == "reference":
        if rank != 0:
            return
        import oracle
        small = cfg.with_layers(1)
        K, V = inputs.make_kv(small, N)
        q1 = qs[0][:1]
        for _ in range(args.warmup):
            oracle.decode_attention(q1, K[:, :, :, :64], V[:, :, :, :64])
        # a step is one layer, or as many of its KV heads as the run's time budget allows (heads are independent)
        t0 = time.perf_counter()
        oracle.decode_attention(q1, K, V)
        t_layer = time.perf_counter() - t0
        share = REFERENCE_BUDGET_S / max(1, args.steps + args.warmup)
        heads = cfg.Hkv if share >= t_layer else max(1, int(cfg.Hkv * share / t_layer))
        G = cfg.Hq // cfg.Hkv
        q1, K, V = (np.ascontiguousarray(q1[:, :, :G * heads]), np.ascontiguousarray(K[:, :, :heads]),
                    np.ascontiguousarray(V[:, :, :heads]))
        times = []
        for _ in range(args.steps):
            t0 = time.perf_counter()
            oracle.decode_attention(q1, K, V)
            times.append(time.perf_counter() - t0)
        ms = float(np.mean(times)) * 1e3 * cfg.layers * cfg.Hkv / heads
        print(json.dumps({
            "impl": "reference", "metric": "decode_tokens_per_s", "value": cfg.batch * 1e3 / ms, "unit": "tokens/s", "n_gpus": 1,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": {"workload": workload},
            "cpu_baseline": {"value": cfg.batch * 1e3 / ms, "unit": "tokens/s", "cores": 1, "kind": "oracle",
                             "sample": f"{heads} of {cfg.Hkv} KV heads of 1 of {cfg.layers} layers per step, extrapolated"},
            "e2e": {"value": cfg.batch * 1e3 / ms, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return

    import torch
    import torch.distributed as dist
    from paper_2410_01518_b200 import ipot

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the compression path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32

    def dev(a):
        t = torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).cuda()
        return t.view(tdt) if a.dtype == np.uint16 else t

    h = ipot.ipot_create_ex(cfg.pot_size, cfg.keep, cfg.layers, cfg.Hq, cfg.Hkv, cfg.d, batch=cfg.batch,
                            dtype=ipot.IPOT_BF16 if cfg.dtype == "bf16" else ipot.IPOT_F32, nuc_slots=cfg.nuc_slots, max_cap_rows=1)
    stream = torch.cuda.current_stream()
    ipot.ipot_set_stream(h, stream.cuda_stream)
    ipot.ipot_set_scorer(h, SCORERS[args.scorer])
    tensor_path = args.scorer != "simt" and cfg.dtype == "bf16" and cfg.d in (64, 128)
    K, V = inputs.make_kv(cfg, N)
    ipot.ipot_append_chunk(h, dev(K), dev(V), N)
    dq = [dev(a) for a in qs]
    hq = [torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory() for a in qs]
    stage_q = torch.empty_like(dq[0])
    out = torch.empty((cfg.layers, cfg.batch, cfg.Hq, cfg.d), device="cuda")
    out_host = torch.empty(out.shape, dtype=torch.float32).pin_memory()
    pot_bytes = 2 * cfg.units * N * cfg.d * cfg.elem_bytes
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda") if pot_bytes <= 126e6 else None

    def step_dev(i):
        if flush is not None:
            flush.add_(1)
        ipot.ipot_decode_attention(h, dq[i % RING], out)

    def step_host(i):
        (stage_q.view(torch.int16) if cfg.dtype == "bf16" else stage_q).copy_(hq[i % RING], non_blocking=True)
        ipot.ipot_decode_attention(h, stage_q, out)
        out_host.copy_(out, non_blocking=True)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(step, steps, warmup, sampler=None):
        for i in range(warmup):
            step(i)
        barrier()
        if sampler:
            sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0 = ipot.ipot_launch_count(h)
        e0.record(stream)
        for i in range(steps):
            step(warmup + i)
        e1.record(stream)
        barrier()
        clocks = sampler.stop() if sampler else None
        rate, ms_step = whole_job_rate(e0.elapsed_time(e1), steps, world, "cuda")
        return rate * cfg.batch, ms_step, ipot.ipot_launch_count(h) - l0, clocks

    value, ms_step, launches, clocks = timed(step_dev, args.steps, args.warmup, ClockSampler(local))
    e2e_value, _, _, _ = timed(step_host, max(3, min(args.steps, 200)), 3)
    assert ipot.ipot_sync_status(h) == 0, "device status is not clean"
    pk = peaks()
    algo = pot_bytes + cfg.layers * cfg.batch * cfg.Hq * cfg.d * (cfg.elem_bytes + 4)   # K and V once, q in, out
    roof = {"kernel": "decode_attn_mma_kernel" if tensor_path else "decode_attn_kernel", "bound": "hbm", "achieved": algo / (ms_step * 1e-3) / 1e9, "peak": pk["hbm_gbs"],
            "unit": "GB/s", "peak_source": pk["source"], "traffic": None}
    roof["frac"] = roof["achieved"] / roof["peak"]
    line = {
        "metric": "decode_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload, "l2": "inputs_larger_than_l2" if flush is None else "l2_flushed_between_steps"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": qs[0].nbytes, "d2h_bytes_per_step": out_host.numel() * 4},
        "gpu_launches": launches, "roofline": roof,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        t0 = time.perf_counter()
        oracle.decode_attention(qs[0][:1], K[:1], V[:1])
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": cfg.batch / (dt * cfg.layers), "unit": "tokens/s", "cores": 1, "kind": "oracle",
                                "sample": f"1 of {cfg.layers} layers in {dt:.2f} s, extrapolated"}
    if rank == 0:
        print(json.dumps(line))
    ipot.ipot_destroy(h)
    if world > 1:
        dist.destroy_process_group()


def run_novelty(args):
    """The novelty producer alone: a step turns one chunk's logits into per-token novelty scores."""
    V, n = NOVELTY_WORKLOADS[args.workload]
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    workload = f"token novelty of {n} new tokens over a {V}-word vocabulary (bf16 logits)"
    if args.impl == "reference":
        if rank != 0:
            return
        import oracle
        sample = max(1, min(128, int(128 * (REFERENCE_BUDGET_S / max(1, args.steps + args.warmup)) / (0.02 * V / 32000))))
        z, lab = inputs.make_logits(inputs.SEED_BASE + V, sample, V, "bf16", 0)
        zw = inputs.widen(z, "bf16")
        for _ in range(args.warmup):
            oracle.token_novelty(zw[:8], lab[:8])
        times = []
        for _ in range(args.steps):
            t0 = time.perf_counter()
            oracle.token_novelty(zw, lab)
            times.append(time.perf_counter() - t0)
        ms = float(np.mean(times)) * 1e3 * n / sample
        value = n * 1e3 / ms
        print(json.dumps({
            "impl": "reference", "metric": "nuc_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": 1,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": {"workload": workload},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": 1, "kind": "oracle",
                             "sample": f"{sample} of {n} rows per step, extrapolated"},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return

    import torch
    import torch.distributed as dist
    from paper_2410_01518_b200 import ipot

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the compression path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    ring = [inputs.make_logits(inputs.SEED_BASE + V, n, V, "bf16", c) for c in range(RING)]  # > L2 in total
    dz = [torch.from_numpy(z.view(np.int16)).cuda().view(torch.bfloat16) for z, _ in ring]
    dl = [torch.from_numpy(lab).cuda() for _, lab in ring]
    hz = [torch.from_numpy(z.view(np.int16)).pin_memory() for z, _ in ring]
    hl = [torch.from_numpy(lab).pin_memory() for _, lab in ring]
    stage_z, stage_l = torch.empty_like(dz[0]), torch.empty_like(dl[0])
    aux = torch.zeros((1, 2 * n), device="cuda")
    aux_host = torch.empty((n,), dtype=torch.float32).pin_memory()
    h = ipot.ipot_create_ex(2 * n, n, 1, 8, 8, 128, batch=1, dtype=ipot.IPOT_BF16, nuc_slots=n // 2, max_cap_rows=1)
    stream = torch.cuda.current_stream()
    ipot.ipot_set_stream(h, stream.cuda_stream)

    def step_dev(i):
        ipot.ipot_nuc_scores(h, dz[i % RING], ipot.IPOT_BF16, V, dl[i % RING], n, V, aux, 2 * n, n)

    def step_host(i):
        stage_z.view(torch.int16).copy_(hz[i % RING], non_blocking=True)
        stage_l.copy_(hl[i % RING], non_blocking=True)
        ipot.ipot_nuc_scores(h, stage_z, ipot.IPOT_BF16, V, stage_l, n, V, aux, 2 * n, n)
        aux_host.copy_(aux[0, n:], non_blocking=True)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(step, steps, warmup, sampler=None):
        for i in range(warmup):
            step(i)
        barrier()
        if sampler:
            sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0 = ipot.ipot_launch_count(h)
        e0.record(stream)
        for i in range(steps):
            step(warmup + i)
        e1.record(stream)
        barrier()
        clocks = sampler.stop() if sampler else None
        rate, ms_step = whole_job_rate(e0.elapsed_time(e1), steps, world, "cuda")
        return rate * n, ms_step, ipot.ipot_launch_count(h) - l0, clocks

    value, ms_step, launches, clocks = timed(step_dev, args.steps, args.warmup, ClockSampler(local))
    e2e_value, _, _, _ = timed(step_host, max(3, min(args.steps, 50)), 3)
    assert ipot.ipot_sync_status(h) == 0, "device status is not clean"
    pk = peaks()
    algo = n * V * 2 + n * 4 + n * 4   # logits once + labels + novelty out
    roof = {"kernel": "novelty_partial_kernel", "bound": "hbm", "achieved": algo / (ms_step * 1e-3) / 1e9,
            "peak": pk["hbm_gbs"], "unit": "GB/s", "peak_source": pk["source"], "traffic": None,
            "note": "duration = the whole step (all launches of one call)"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    line = {
        "metric": "nuc_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload, "l2": "inputs_larger_than_l2", "ring": RING},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": n * V * 2 + n * 4, "d2h_bytes_per_step": n * 4},
        "gpu_launches": launches, "roofline": roof,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        sample = 256
        zw = inputs.widen(ring[0][0][:sample], "bf16")
        t0 = time.perf_counter()
        oracle.token_novelty(zw, ring[0][1][:sample])
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": sample / dt, "unit": "tokens/s", "cores": 1, "kind": "oracle",
                                "sample": f"{sample} of {n} rows of one step in {dt:.2f} s"}
    if rank == 0:
        print(json.dumps(line))
    ipot.ipot_destroy(h)
    if world > 1:
        dist.destroy_process_group()


def config_dict(cfg, n_new, N, cap_keys=False, rope=False):
    return {"workload": f"configs[{cfg.cfg_id - 1}] {cfg.name}: one CCD cycle per step "
                        f"(append {n_new} rows, distil {N} -> {cfg.keep})"
                        + ("; CaP keys inside the softmax" if cap_keys else "") + ("; rotary mode" if rope else ""),
            "layers": cfg.layers, "batch": cfg.batch, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "d": cfg.d,
            "pot_size": cfg.pot_size, "keep": cfg.keep, "nuc_slots": cfg.nuc_slots, "cap_rows": cfg.cap_rows,
            "units": cfg.units, "l2": "inputs_larger_than_l2" if cfg.units * N * cfg.d * cfg.elem_bytes * 2 > 126e6
            else "l2_flushed_between_steps"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=sorted(WORKLOADS) + sorted(NOVELTY_WORKLOADS) + sorted(DECODE_WORKLOADS))
    ap.add_argument("--scorer", default="auto", choices=sorted(SCORERS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cap-keys", action="store_true",
                    help="score with the CaP's own keys inside the softmax (the Appendix B listing read literally)")
    ap.add_argument("--rope", action="store_true",
                    help="context-reset rotary mode: unrotated keys in the pot, the row movers keep a rotated copy")
    ap.add_argument("--layers", type=int, default=0, help="override the workload's layer count (profiling small cases)")
    ap.add_argument("--append", default="deferred", choices=["deferred", "eager"],
                    help="deferred: the chunk stays in the caller's buffers, the scorer reads its keys there and the "
                         "compaction fetches the surviving rows (ipot_set_deferred_append); eager: copied at append")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.workload in NOVELTY_WORKLOADS:
        run_novelty(args)
        return
    if args.workload in DECODE_WORKLOADS:
        run_decode(args)
        return
    cfg = inputs.CONFIGS[WORKLOADS[args.workload]]
    if args.layers > 0:
        cfg = cfg.with_layers(args.layers)
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import torch.distributed as dist
    from paper_2410_01518_b200 import ipot

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the compression path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    n_new, N = workload_shape(cfg)
    ring, K0, V0 = gen_ring(cfg, n_new, args.cap_keys)
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32

    def dev(a):
        t = torch.from_numpy(a.view(np.int16) if cfg.dtype == "bf16" and a.dtype == np.uint16 else a).cuda()
        return t.view(tdt) if a.dtype == np.uint16 else t

    def pin(a):
        return torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()

    dring = [{k: dev(v) for k, v in t.items()} for t in ring]
    hring = [{k: pin(v) for k, v in t.items()} for t in ring]
    K0d, V0d = dev(K0), dev(V0)
    idx_host = torch.empty((cfg.units, cfg.keep), dtype=torch.int32).pin_memory()

    h = ipot.ipot_create_ex(cfg.pot_size, cfg.keep, cfg.layers, cfg.Hq, cfg.Hkv, cfg.d, batch=cfg.batch,
                            dtype=ipot.IPOT_BF16 if cfg.dtype == "bf16" else ipot.IPOT_F32,
                            nuc_slots=cfg.nuc_slots, max_cap_rows=cfg.cap_rows)
    ipot.ipot_set_scorer(h, SCORERS[args.scorer])
    if args.rope:
        rope_tables = [dev(a) for a in inputs.make_rope_table(cfg.pot_size, cfg.d, cfg.dtype)]
        ipot.ipot_enable_rope(h, rope_tables[0], rope_tables[1], ipot.IPOT_ROPE_HALF)
    stream = torch.cuda.current_stream()
    ipot.ipot_set_stream(h, stream.cuda_stream)
    ipot.ipot_set_deferred_append(h, args.append == "deferred")
    ipot.ipot_append_chunk(h, K0d, V0d, cfg.keep)

    small_l2 = cfg.units * N * cfg.d * cfg.elem_bytes * 2 <= 126e6
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda") if small_l2 else None

    def step_dev(i):
        t = dring[i % RING]
        if flush is not None:
            flush.add_(1)
        ipot.ipot_append_chunk(h, t["K"], t["V"], n_new)
        if args.cap_keys:
            ipot.ipot_score_and_compress_cap(h, t["Q"], t["K_cap"], cfg.cap_rows, t["aux"])
        else:
            ipot.ipot_score_and_compress(h, t["Q"], cfg.cap_rows, t["aux"])

    def step_host(i):
        t = hring[i % RING]
        ipot.ipot_append_chunk_host(h, t["K"], t["V"], n_new)
        if args.cap_keys:
            ipot.ipot_score_and_compress_cap_host(h, t["Q"], t["K_cap"], cfg.cap_rows, t["aux"], idx_host)
        else:
            ipot.ipot_score_and_compress_host(h, t["Q"], cfg.cap_rows, t["aux"], idx_host)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(step, steps, warmup, sampler=None, repeats=1):
        """Exactly `steps` steps between two events, bracketed by barrier + synchronize; with repeats > 1 the same
        region is run that many times (each bracketed the same way) and the median region counts."""
        for i in range(warmup):
            step(i)
        barrier()
        if sampler:
            sampler.start()
        l0 = ipot.ipot_launch_count(h)
        times = []
        for r in range(repeats):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for i in range(steps):
                step(warmup + r * steps + i)
            e1.record(stream)
            barrier()
            times.append(e0.elapsed_time(e1))
        clocks = sampler.stop() if sampler else None
        rate, ms_step = whole_job_rate(float(np.median(times)), steps, world, "cuda")
        return rate, ms_step, (ipot.ipot_launch_count(h) - l0) // repeats, clocks

    # untimed pre-heat: the first few hundred milliseconds after idle run at lower memory throughput (the compaction
    # kernel takes 105 us averaged over the first 0.1 s of steps, 91 us over 0.3 s, 82 us afterwards)
    t_end = time.perf_counter() + PREHEAT_S
    i = 0
    while time.perf_counter() < t_end:
        for _ in range(50):
            step_dev(i)
            i += 1
        torch.cuda.synchronize()
    # device-resident inputs: the headline value over exactly K steps, no instrumentation inside the region
    # a short region (few steps) is repeated so that the clock sampler sees MIN_SAMPLED_S of it; the median region counts
    _, ms_probe, _, _ = timed(step_dev, 20, 0)
    repeats = int(min(2000, max(1, np.ceil(MIN_SAMPLED_S * 1e3 / (ms_probe * args.steps)))))
    if world > 1:   # every rank must run the same number of regions
        r_t = torch.tensor([repeats], device="cuda")
        dist.all_reduce(r_t, op=dist.ReduceOp.MAX)
        repeats = int(r_t.item())
    sampler = ClockSampler(local)
    value, ms_step, launches, clocks = timed(step_dev, args.steps, args.warmup, sampler, repeats)
    assert ipot.ipot_sync_status(h) == 0, "device status is not clean"
    # the same K steps once more with the library's per-kernel CUDA events (they serialise the kernel boundaries,
    # which costs a few microseconds per step: reported beside the headline, not as it)
    ipot.ipot_set_profiling(h, 1)
    for i in range(3):
        step_dev(i)
    torch.cuda.synchronize()
    ipot.ipot_kernel_ms(h)  # drop the warm-up cycles from the per-kernel means
    _, ms_step_events, _, _ = timed(step_dev, min(args.steps, 2000), 0)   # the library keeps events for 2048 cycles
    kms, kcycles, scorer_used = ipot.ipot_kernel_ms(h)
    ipot.ipot_set_profiling(h, 0)
    assert ipot.ipot_sync_status(h) == 0, "device status is not clean"
    # the same K steps with the other append mode, for comparison
    ipot.ipot_set_deferred_append(h, args.append != "deferred")
    _, ms_step_other, _, _ = timed(step_dev, args.steps, 3)
    ipot.ipot_set_deferred_append(h, args.append == "deferred")
    assert ipot.ipot_sync_status(h) == 0, "device status is not clean"

    # end to end: host (pinned) buffers in, index lists out, copies inside the timed region
    e2e_steps = max(3, min(args.steps, 50))
    e2e_value, _, _, _ = timed(step_host, e2e_steps, 3)
    assert ipot.ipot_sync_status(h) == 0
    h2d = sum(v.numel() * v.element_size() for v in hring[0].values())
    d2h = idx_host.numel() * 4

    # roofline of the dominant kernel
    pk = peaks()
    units, e, d, M = cfg.units, cfg.elem_bytes, cfg.d, cfg.G * cfg.cap_rows
    score_bytes = units * (N * d * e + M * d * e + 4 * N)      # K once + Q + scores out
    score_flops = 2.0 * units * M * N * d                      # one pass (a second sweep is overhead, not algorithm)
    # K and V, read + write, all kept rows; in rotary mode the rotated copy of K is written as well
    compact_bytes = units * (5 if args.rope else 4) * cfg.keep * d * e
    names = ["nuc_rank", "cap_score", "select", "compact"]
    # the dominant kernel; scoring and compaction are close, scoring is named unless compaction is clearly longer
    dom = 3 if kms[3] > 1.05 * kms[1] else 1
    score_gbs = score_bytes / (kms[1] * 1e-3) / 1e9
    score_tflops = score_flops / (kms[1] * 1e-3) / 1e12
    if names[dom] == "compact":
        roof = {"kernel": "compact_kernel", "bound": "hbm", "achieved": compact_bytes / (kms[3] * 1e-3) / 1e9,
                "peak": pk["hbm_gbs"], "unit": "GB/s"}
    else:
        # which roof binds Eq. 2 on this shape: reading K once at the copy rate, or 2 M N d flops per unit at the
        # sustained bf16 rate (the fp32-FMA scorer is not a tensor-core kernel: its line is reported against HBM)
        t_hbm = score_bytes / (pk["hbm_gbs"] * 1e9)
        t_tensor = score_flops / (pk["bf16_tflops"] * 1e12) if cfg.dtype == "bf16" and scorer_used != 1 else 0.0
        kernel = SCORER_KERNELS.get(scorer_used, "cap_score")
        if t_tensor > t_hbm:
            roof = {"kernel": kernel, "bound": "tensor", "achieved": score_tflops, "peak": pk["bf16_tflops"], "unit": "TFLOP/s"}
        else:
            roof = {"kernel": kernel, "bound": "hbm", "achieved": score_gbs, "peak": pk["hbm_gbs"], "unit": "GB/s"}
        roof["roof_us"] = {"hbm": round(t_hbm * 1e6, 2), "tensor": round(t_tensor * 1e6, 2)}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["peak_source"] = pk["source"]
    if roof["unit"] == "GB/s":
        roof["frac_of_nominal_8tbs"] = roof["achieved"] / 8000.0   # the HBM3e data-sheet figure, for context
    # DRAM bytes of one launch of the dominant kernel, from the committed ncu captures (profiles/dram_traffic.txt: measured
    # on a few layers of the same shape and scaled by the units, which is how the traffic grows); null if no capture
    # of this kernel and shape is on record
    tkey = {1: "simt", 2: "cap_score_tc", 3: "warp_mma", 4: "cap_score_ts"}.get(scorer_used, "?") if dom == 1 else "compact"
    roof["traffic"] = None if (args.cap_keys or args.rope) else recorded_traffic(tkey, f"N{N}_M{M}_d{d}_{cfg.dtype}", units)
    roof["kernel_ms"] = dict(zip(names, [round(x, 5) for x in kms]))
    roof["cycles_averaged"] = kcycles
    roof["cap_score_gbs"] = score_gbs
    roof["cap_score_tflops"] = score_tflops
    roof["cap_score_frac_of_hbm_peak"] = score_gbs / pk["hbm_gbs"]
    roof["cap_score_frac_of_bf16_sustained"] = score_tflops / pk["bf16_tflops"]
    roof["compact_gbs"] = compact_bytes / (kms[3] * 1e-3) / 1e9
    roof["compact_frac_of_hbm_peak"] = roof["compact_gbs"] / pk["hbm_gbs"]
    # the whole step against the copy rate: algorithmic bytes of scoring + compaction (+ the append's copy when it is
    # made at append time) over the step's time
    step_bytes = score_bytes + compact_bytes + (0 if args.append == "deferred" else units * 4 * n_new * d * e)
    roof["step_gbs"] = step_bytes / (ms_step * 1e-3) / 1e9
    roof["step_frac_of_hbm_peak"] = roof["step_gbs"] / pk["hbm_gbs"]

    line = {
        "metric": "ccd_cycles_per_s", "value": value, "unit": "cycles/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": config_dict(cfg, n_new, N, args.cap_keys, getattr(args, "rope", False)),
        "preheat_s": PREHEAT_S,   # untimed running before the warm-up steps: the value is a warm steady state
        "append": ("deferred: the chunk stays in the caller's device buffers, the scorer reads its keys there, "
                   "the compaction copies the surviving rows into the pot" if args.append == "deferred"
                   else "eager: all rows copied into the pot by the append call"),
        "repeats": repeats,       # timed regions of `steps` steps each; ms_per_step is the median region's
        "pot_tokens_per_s": value * N * cfg.batch,
        "layer_cycles_per_s": value * cfg.layers,
        "ms_per_step_with_kernel_events": ms_step_events,
        ("ms_per_step_eager_append" if args.append == "deferred" else "ms_per_step_deferred_append"): ms_step_other,
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "cycles/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps},
        "gpu_launches": launches,
        "roofline": roof,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n_sample = min(cfg.units, 256)
        v, dt, n_units, threads = cpu_baseline(cfg, ring, K0, V0, n_sample, rope=args.rope)
        line["cpu_baseline"] = {"value": v, "unit": "cycles/s", "cores": threads, "kind": "oracle",
                                "sample": f"{n_units} of {cfg.units} units of one cycle in {dt:.1f} s; "
                                          f"full-cycle rate extrapolated (units are independent and equal-sized)"}
    ipot.ipot_destroy(h)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
