#!/usr/bin/env python
"""Benchmark of the PAMM hot path on B200: tokens/s per fused Q|K|V layer.

One "step" = one pass of the whole path over one batch of synthetic input:
select generators + compress X (forward), then contract dY + C^T B~ (backward).
Prints ONE JSON line (rank 0).  `--impl reference` times the fp64 CPU oracle on
a bounded sample of the same workload instead.

Multi-GPU (torchrun, one rank per GPU) is data-parallel replicas, as in the
paper's DDP runs: every rank compresses its own tokens with its own generators;
there is no collective on the data path, only the barrier and the max-over-ranks
reduction of the timing.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

METRIC = "PAMM compress + weight-grad tokens/sec per QKV layer; achieved HBM GB/s vs peak"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1400.0      # sustained, inside a long step
NOMINAL_HBM_GBS = 8000.0           # the data-sheet figure the fractions "of nominal" refer to
PROF_EVERY = 16     # one step in PROF_EVERY carries per-kernel CUDA events, another one the stage events;
                    # the rest run event-free, since an event between two kernels serialises their launches
MIN_SAMPLES = 32    # stage / kernel samples behind every reported median; short runs top up after the timed region
TRAFFIC_FILE = ROOT / "profiles" / "dominant_kernel_traffic.txt"


def env_int(name, default):
    try:
        return int(os.environ.get(name, default))
    except ValueError:
        return default


def dist_setup(n_gpus: int, backend: str):
    """Initialise torch.distributed when launched with WORLD_SIZE > 1."""
    import torch.distributed as dist
    world = env_int("WORLD_SIZE", 1)
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend=backend, rank=env_int("RANK", 0), world_size=world)
    return env_int("RANK", 0), world


def aggregate(ms_local: float, tokens_local: int, device="cpu"):
    """(max over ranks of the time, sum over ranks of the tokens); identity on one rank."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms_local, tokens_local
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    n = torch.tensor([tokens_local], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), int(n.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50", "-i", str(self.gpu)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, smax, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            p = [x.strip() for x in line.split(",")]
            if len(p) < 9:
                continue
            try:
                sm.append(float(p[1]))
                smax = float(p[2])
            except ValueError:
                continue
            for nm, v in zip(names, p[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": smax, "samples": len(sm),
                "reasons": sorted(reasons)}


def measured_peaks():
    """(HBM GB/s, sustained dense bf16 TFLOP/s, "measured" | "fallback")."""
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            d = json.loads(p.read_text())
            return float(d["hbm_gbs"]), float(d.get("bf16_tflops_sustained", FALLBACK_BF16_TFLOPS)), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, "fallback"


def ncu_traffic(workload: str, kernel_source: Path):
    """DRAM bytes (read + write) of one launch of the dominant kernel, from the ncu capture summarised under
    profiles/.  A line of the file reads `workload bytes sha256-of-the-kernel-source ...`; the figure is
    reported only while the kernel's source is the one the counters were taken from."""
    import hashlib
    try:
        digest = hashlib.sha256(kernel_source.read_bytes()).hexdigest()[:16]
        for line in TRAFFIC_FILE.read_text().splitlines():
            p = line.split()
            if len(p) >= 3 and not line.startswith("#") and p[0] == workload and p[2] == digest:
                return int(p[1])
    except (OSError, ValueError):
        pass
    return None


def stats(x) -> dict:
    x = np.asarray(x, dtype=np.float64)
    return {"count": int(x.size), "median": float(np.median(x)), "min": float(x.min()), "mean": float(x.mean())}


def algorithmic_bytes(b, n, m, k, e, dw_e=4):
    """Bytes the method itself must move per step (per layer), by stage."""
    return {
        "compress": b * n * e + 8 * b + k * n * e,
        "contract": b * m * e + 8 * b,
        "weight_grad": n * m * dw_e + k * n * e + k * m * 4,
    }


def run_reference(args):
    """The fp64 oracle on host cores, on a bounded sample of the workload."""
    rank = env_int("RANK", 0)
    if rank != 0:
        return
    from oracle import pamm_oracle as orc
    from paper_2506_02939_b200 import synth
    w = synth.WORKLOADS[args.workload]
    k = w.ks[0]
    max_seqs = max(1, min(w.num_seqs, args.ref_tokens // w.seq_len))
    full = synth.make_inputs(args.workload, num_seqs=max_seqs)

    def sample(seqs):
        bs = seqs * w.seq_len
        rng = np.random.default_rng(w.index_seed)
        return full.X[:bs], full.dY[:bs], np.sort(rng.choice(bs, size=min(k, bs), replace=False)).astype(np.int32)

    # size the per-step sample so that all steps fit the time budget: one calibration pass on one sequence
    Xc, dYc, Ic = sample(1)
    orc.pamm(Xc, Ic, dYc)
    t0 = time.perf_counter()
    orc.pamm(Xc, Ic, dYc)
    per_seq = max(1e-6, time.perf_counter() - t0)
    seqs = int(args.ref_budget_s / (max(1, args.steps + args.warmup) * per_seq))
    seqs = max(1, min(max_seqs, seqs))
    X, dY, I = sample(seqs)
    b = X.shape[0]

    def step():
        orc.pamm(X, I, dY)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    val = b * args.steps / dt
    sample = f"first {b} of {w.b} tokens of workload {w.name} per step, k={len(I)}, all stages, fp64"
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{w.name}: b={w.b} n={w.n} m={w.m} k={k} {w.dtype}", "sample": sample},
        "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": orc.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_cuda(args):
    import torch
    from paper_2506_02939_b200 import build as pamm_build, synth
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the PAMM path has no CPU fallback")
    local = env_int("LOCAL_RANK", 0)
    torch.cuda.set_device(local)
    rank, world = dist_setup(args.gpus, "nccl")
    if rank == 0:
        pamm_build.build()
    barrier()
    from paper_2506_02939_b200 import pamm

    w = synth.WORKLOADS[args.workload]
    k = args.k or w.ks[0]
    e = 2 if w.dtype == "bf16" else 4
    dt_code = pamm.BF16 if w.dtype == "bf16" else pamm.F32
    inp = synth.make_inputs(args.workload, seed=w.seed + 7919 * rank)
    b, n, m = inp.b, w.n, w.m
    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32

    def host_tensor(a):
        t = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16) if a.dtype == np.uint16 else torch.from_numpy(a)
        return t.pin_memory()

    Xh, dYh = host_tensor(inp.X), host_tensor(inp.dY)
    X, dY = Xh.cuda(non_blocking=True), dYh.cuda(non_blocking=True)
    dev = X.device
    idx = torch.empty(k, dtype=torch.int32, device=dev)
    C = torch.empty((k, n), dtype=tdt, device=dev)
    invn = torch.empty(2 * k, dtype=torch.float32, device=dev)
    f = torch.empty(b, dtype=torch.int32, device=dev)
    alpha = torch.empty(b, dtype=torch.float32, device=dev)
    Bt = torch.empty((k, m), dtype=torch.float32, device=dev)
    dw_tdt = torch.bfloat16 if args.dw_dtype == "bf16" else torch.float32
    layout = pamm.DW_MN if args.layout == "mn" else pamm.DW_NM
    dW = torch.empty((m, n) if layout == pamm.DW_MN else (n, m), dtype=dw_tdt, device=dev)
    ws = pamm.alloc_workspace(pamm.WS_CONTRACT, b, n, m, k, dt_code, dev)
    sp = pamm.alloc_workspace(pamm.WS_COMPRESS, b, n, m, k, dt_code, dev)     # the forward's counts of f, for the backward's sort
    stream = torch.cuda.current_stream()

    eps = args.eps
    dropped = torch.zeros(1, dtype=torch.int32, device=dev)

    # the arguments of the two fused calls are marshalled once (a fresh index seed per step, 64 of them in turn):
    # at the small workloads a step is a few microseconds of GPU work and Python's argument handling would dominate
    SEEDS = 64
    fwd_calls = [pamm.prepared(pamm.compress_fused, X, k, w.index_seed + s, idx_out=idx, C=C, c_invnorm=invn, f=f, alpha=alpha,
                               sort_products=sp, stream=stream) for s in range(SEEDS)] if eps is None else None
    bwd_call = pamm.prepared(pamm.contract_weight_grad, C, f, alpha, dY, Btilde=Bt, dW=dW, layout=layout, sort_products=sp,
                             workspace=ws, stream=stream) if eps is None else None

    def forward(seed):
        if eps is None:
            fwd_calls[(seed - w.index_seed) % SEEDS]()
        else:     # neighbourhood condition (Eq. 2): select, then compress with the row-norm warps
            pamm.select_generators(X, k, seed, idx_out=idx, C=C, c_invnorm=invn, stream=stream)
            pamm.compress_eps(X, C, invn, eps, f=f, alpha=alpha, dropped=dropped, sort_products=sp, stream=stream)

    def backward():
        if eps is None:
            bwd_call()
        else:     # beta = b / (b - eta) applied by the product's epilogue (Eq. 4-5)
            pamm.contract(f, alpha, dY, k, Btilde=Bt, sort_products=sp, workspace=ws, stream=stream)
            pamm.weight_grad_beta(C, Bt, b, dropped, dW=dW, layout=layout, stream=stream)

    def step(seed):
        forward(seed)
        backward()

    for s in range(args.warmup):
        step(w.index_seed + s)
    torch.cuda.synchronize()
    status = pamm.last_device_status()
    if status != pamm.OK:
        raise SystemExit(f"device status after warm-up: {pamm.status_string(status)}")

    # ---- timed region: device-resident inputs ----------------------------------
    K = args.steps
    KINDS = (pamm.PROF_COMPRESS, pamm.PROF_CONTRACT, pamm.PROF_WEIGHT_GRAD)

    # Steps of the timed region that carry events: one in PROF_EVERY for the kernels and as many for
    # the stages; a run too short for that carries one kernel step, its last, and no stage step.
    if K >= 4 * PROF_EVERY:
        kernel_at = set(range(0, K, PROF_EVERY))
        stage_at = set(range(PROF_EVERY // 2, K, PROF_EVERY))
    else:
        kernel_at, stage_at = {K - 1}, set()
    event_pool = []

    def new_event():
        if event_pool:
            return event_pool.pop()
        e = torch.cuda.Event(enable_timing=True)
        e.record(stream)          # creates the underlying CUDA event, whose handle the library records later
        return e

    # the events the timed region will use exist before it starts
    event_pool.extend([new_event() for _ in range(2 * len(KINDS) * len(kernel_at))])

    def kernel_step(seed):
        """One step with an event pair around each step's main kernel."""
        pairs = {kind: (new_event(), new_event()) for kind in KINDS}
        for kind in KINDS:
            pamm.set_profile_events(kind, *pairs[kind])
        step(seed)
        for kind in KINDS:
            pamm.set_profile_events(kind, None, None)
        return pairs

    def staged_step(seed):
        """One step with events around the forward and the backward stage."""
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record(stream)
        forward(seed)
        e[1].record(stream)
        backward()
        e[2].record(stream)
        return e

    # event pairs on a few steps only: an event between two kernels serialises them,
    # the other steps keep the back-to-back launch overlap
    kernel_samples, stage_samples = [], []
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    launches0 = pamm.launch_count()
    barrier()
    torch.cuda.synchronize()
    sampler.start()
    t_begin.record(stream)
    for s in range(K):
        if s in kernel_at:
            kernel_samples.append(kernel_step(w.index_seed + s))
        elif s in stage_at:
            stage_samples.append(staged_step(w.index_seed + s))
        else:
            step(w.index_seed + s)
    t_end.record(stream)
    torch.cuda.synchronize()
    launches = pamm.launch_count() - launches0
    barrier()
    in_region = (len(kernel_samples), len(stage_samples))
    # a short run yields too few samples for a median: top them up in an untimed pass over the same steps
    extra = 0
    while len(kernel_samples) < MIN_SAMPLES or len(stage_samples) < MIN_SAMPLES:
        kernel_samples.append(kernel_step(w.index_seed + extra))
        step(w.index_seed + extra)
        stage_samples.append(staged_step(w.index_seed + extra))
        step(w.index_seed + extra)
        extra += 1
    torch.cuda.synchronize()

    # each stage repeated back to back (untimed region): its throughput when the launches overlap as they do
    # inside a step, without the event records that bracket a single stage above
    def repeat_ms(fn, reps=64):
        for s in range(4):
            fn(w.index_seed + s)
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for s in range(reps):
            fn(w.index_seed + s)
        z.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(z) / reps

    fwd_rep = repeat_ms(forward)
    bwd_rep = repeat_ms(lambda s: backward())
    forward(w.index_seed)          # leave (C, f, alpha) of a forward pass behind, as after a step

    # the read-only ceiling (untimed region): passes that only read dY or X, with plain loads and with the bulk-copy
    # ring of the contraction's main pass, in natural row order and in the contraction's order (rows sorted by f)
    def probe_gbs(kind, data, order=None, reps=12):
        word = torch.empty(1, dtype=torch.int32, device=dev)
        for _ in range(2):
            pamm.probe_read(kind, data, order=order, sum32=word, stream=stream)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
        ev[0].record(stream)
        for r in range(reps):
            pamm.probe_read(kind, data, order=order, sum32=word, stream=stream)
            ev[r + 1].record(stream)
        torch.cuda.synchronize()
        ms = float(np.median([ev[r].elapsed_time(ev[r + 1]) for r in range(reps)]))
        return data.shape[0] * data.shape[1] * data.element_size() / (ms * 1e-3) / 1e9

    read_ceiling = None
    if m * e <= 24576 and n * e <= 24576 and (m * e) % 16 == 0 and (n * e) % 16 == 0:
        sorted_rows = torch.sort(f.to(torch.int64), stable=True).indices.to(torch.int32)
        read_ceiling = {"unit": "GB/s",
                        "dY_plain_loads": probe_gbs(pamm.PROBE_SUM, dY),
                        "dY_bulk_rows_natural_order": probe_gbs(pamm.PROBE_ROWS, dY),
                        "dY_bulk_rows_sorted_by_f": probe_gbs(pamm.PROBE_ROWS, dY, sorted_rows),
                        # X is dense: swept in 12 KB pieces (its own rows are too narrow to keep the ring's bytes in flight)
                        "X_bulk_natural_order": probe_gbs(pamm.PROBE_ROWS, X.reshape(-1, 12288 // e) if X.is_contiguous()
                                                          and X.numel() % (12288 // e) == 0 else X),
                        "note": "load-only passes over the same buffers; the contraction reads dY in the sorted order"}
    covers = "timed region"
    if t_begin.elapsed_time(t_end) < 500.0:
        # a region this short yields too few 50 ms samples: keep sampling over an untimed repeat of the same steps
        covers = "timed region + untimed repeat of it (region shorter than 0.5 s)"
        t_rep = time.perf_counter()
        while time.perf_counter() - t_rep < 0.5:
            for s in range(16):
                step(w.index_seed + s)
            torch.cuda.synchronize()
    clocks = sampler.stop()
    clocks["covers"] = covers
    status = pamm.last_device_status()
    if status != pamm.OK:
        raise SystemExit(f"device status after the timed region: {pamm.status_string(status)}")
    ms_total_local = t_begin.elapsed_time(t_end)
    ms_total, tokens = aggregate(ms_total_local, b * K, device=dev)
    fwd = np.array([e[0].elapsed_time(e[1]) for e in stage_samples])
    bwd = np.array([e[1].elapsed_time(e[2]) for e in stage_samples])
    kern = {kind: np.array([p[kind][0].elapsed_time(p[kind][1]) for p in kernel_samples]) for kind in KINDS}
    sampling = {"kernel_events_in_timed_region": in_region[0], "stage_events_in_timed_region": in_region[1],
                "added_in_untimed_pass_after_it": [len(kernel_samples) - in_region[0], len(stage_samples) - in_region[1]]}

    # ---- end to end through the host-buffer entry point ----------------------------
    arena = pamm.alloc_workspace(pamm.WS_STEP_HOST, b, n, m, k, dt_code, dev)
    dWh = torch.empty((n, m), dtype=torch.float32).pin_memory()
    Ke = max(3, min(K, args.e2e_steps))
    for s in range(2):
        pamm.qkv_step_host(Xh, dYh, k, w.index_seed + s, dWh, arena, stream=stream)
    torch.cuda.synchronize()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for s in range(Ke):
        pamm.qkv_step_host(Xh, dYh, k, w.index_seed + s, dWh, arena, stream=stream)
    e1.record(stream)
    torch.cuda.synchronize()
    barrier()
    ms_e2e, tokens_e2e = aggregate(e0.elapsed_time(e1), b * Ke, device=dev)
    checksum = float(dWh.double().abs().sum())

    if rank != 0:
        return
    peak, peak_tf, peak_kind = measured_peaks()
    dw_e = 2 if args.dw_dtype == "bf16" else 4
    ab = algorithmic_bytes(b, n, m, k, e, dw_e)
    # rows whose alpha is zero are left out of the contraction's sorted order and never read
    rows_read = int((alpha != 0).sum().item())
    ab["contract"] = rows_read * m * e + 8 * b
    st_f, st_b = stats(fwd), stats(bwd)
    st_k = {"compress": stats(kern[pamm.PROF_COMPRESS]), "contract_main": stats(kern[pamm.PROF_CONTRACT]),
            "weight_grad": stats(kern[pamm.PROF_WEIGHT_GRAD])}
    t_contract = st_k["contract_main"]["median"] * 1e-3
    achieved = ab["contract"] / t_contract / 1e9

    def frac(gbs):
        return {"gbs": gbs, "of_measured": gbs / peak, "of_nominal_8TBs": gbs / NOMINAL_HBM_GBS}

    stages = {
        "sampling": sampling,
        "compress_ms": st_f, "contract_wgrad_ms": st_b,
        "compress_tokens_per_s": b / (st_f["median"] * 1e-3),
        "contract_wgrad_tokens_per_s": b / (st_b["median"] * 1e-3),
        "compress_stage": frac(ab["compress"] / (st_f["median"] * 1e-3) / 1e9),
        "compress_stage_best": frac(ab["compress"] / (st_f["min"] * 1e-3) / 1e9),
        "contract_wgrad_stage": frac((ab["contract"] + ab["weight_grad"]) / (st_b["median"] * 1e-3) / 1e9),
        "contract_wgrad_stage_best": frac((ab["contract"] + ab["weight_grad"]) / (st_b["min"] * 1e-3) / 1e9),
        "compress_stage_repeated_back_to_back": dict(ms=fwd_rep, **frac(ab["compress"] / (fwd_rep * 1e-3) / 1e9)),
        "contract_wgrad_stage_repeated_back_to_back": dict(ms=bwd_rep, **frac((ab["contract"] + ab["weight_grad"]) / (bwd_rep * 1e-3) / 1e9)),
        "whole_step": frac(sum(ab.values()) / (ms_total / K * 1e-3) / 1e9),
        "kernel_ms": st_k,
        "kernel": {"compress": frac(ab["compress"] / (st_k["compress"]["median"] * 1e-3) / 1e9),
                   "contract_main": frac(achieved),
                   "weight_grad": frac(ab["weight_grad"] / (st_k["weight_grad"]["median"] * 1e-3) / 1e9)},
        "algorithmic_bytes": ab,
    }
    stages["compress_stage_frac"] = stages["compress_stage"]["of_measured"]
    stages["contract_wgrad_stage_frac"] = stages["contract_wgrad_stage"]["of_measured"]
    saved = pamm.saved_bytes(b, n, k, dt_code)
    # the dominant kernel: the contract main pass (HBM-bound), except where the scoring contraction is heavy enough to
    # make compress both the longest kernel and tensor-bound (2 b k n flops against b n e bytes: k above the ridge)
    t_compress = st_k["compress"]["median"] * 1e-3
    flops = 2.0 * b * k * n
    if w.dtype == "bf16" and t_compress > t_contract and flops / ab["compress"] > peak_tf * 1e12 / (peak * 1e9):
        tf = flops / t_compress / 1e12
        roofline = {"bound": "tensor", "kernel": "compress_pair_kernel (scoring X C^T + argmax on pairs of CTAs)", "achieved": tf, "peak": peak_tf,
                    "peak_source": f"of {peak_kind} (sustained bf16)", "unit": "TFLOP/s", "frac": tf / peak_tf, "traffic": None,
                    "algorithmic_flops": flops, "samples": st_k["compress"]["count"]}
    else:
        roofline = {"bound": "hbm", "kernel": "contract_stream_kernel (contract main pass)", "achieved": achieved, "peak": peak,
                    "peak_source": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
                    "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                    "traffic": ncu_traffic(w.name, ROOT / "paper_2506_02939_b200" / "csrc" / "contract_stream.cuh")
                    if k == w.ks[0] and args.eps is None else None,
                    "algorithmic_bytes": ab["contract"], "samples": st_k["contract_main"]["count"],
                    "achieved_best": ab["contract"] / (st_k["contract_main"]["min"] * 1e-3) / 1e9}
        if read_ceiling:
            roofline["frac_of_read_ceiling_same_order"] = achieved / read_ceiling["dY_bulk_rows_sorted_by_f"]

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        from oracle import pamm_oracle as orc
        seqs = max(1, min(w.num_seqs, args.ref_tokens // w.seq_len))
        bs = seqs * w.seq_len
        Xs, dYs = inp.X[:bs], inp.dY[:bs]
        I = pamm.draw_indices_host(bs, min(k, bs), w.index_seed).numpy()
        t0 = time.perf_counter()
        reps = 0
        while reps < 1 or (time.perf_counter() - t0 < 10.0 and reps < 50):
            orc.pamm(Xs, I, dYs)
            reps += 1
        dt = time.perf_counter() - t0
        cpu = {"value": bs * reps / dt, "unit": "tokens/s", "cores": orc.num_threads(), "kind": "oracle",
               "sample": f"first {bs} of {b} tokens, k={min(k, bs)}, all stages, {reps} passes in {dt:.1f} s"}

    line = {
        "metric": METRIC, "value": tokens / (ms_total * 1e-3), "unit": "tokens/s", "n_gpus": world,
        "steps": K, "warmup": args.warmup, "ms_per_step": ms_total / K, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": f"{w.name}: X {w.dtype} b={b} n={n}, dY b x m={m}, k={k}, per rank"
                               + ("" if eps is None else f", eps={eps} (dropped {int(dropped.item())} rows)")
                               + ("" if args.dw_dtype == "f32" and args.layout == "nm" else f", dW {args.dw_dtype} {args.layout}"),
                   "l2": "inputs exceed L2 (X %.0f MiB, dY %.0f MiB per step)" % (b * n * e / 2**20, b * m * e / 2**20)
                   if b * n * e > 126 * 2**20 else "inputs fit L2: warm-cache numbers",
                   "parallelism": f"replicas x{world}"},
        "roofline": roofline,
        "cpu_baseline": cpu,
        "e2e": {"value": tokens_e2e / (ms_e2e * 1e-3), "unit": "tokens/s",
                "h2d_bytes_per_step": int(Xh.numel() * e + dYh.numel() * e), "d2h_bytes_per_step": int(dWh.numel() * 4),
                "steps": Ke, "ms_per_step": ms_e2e / Ke, "checksum": checksum},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "stages": stages,
        "read_ceiling": read_ceiling,
        "rows_with_nonzero_alpha": rows_read,
        "memory_saved": saved,
    }
    print(json.dumps(line), flush=True)


def run_forward(args):
    """The forward pass of the layer (Algorithm 2) with the compression fused into the product:
    time of pamm_linear_forward against the same kernel without generators plus the stand-alone
    compression, and the tensor roofline fraction.  torch's own GEMM is timed as context only."""
    import torch
    from paper_2506_02939_b200 import build as pamm_build, synth
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the PAMM path has no CPU fallback")
    torch.cuda.set_device(env_int("LOCAL_RANK", 0))
    pamm_build.build()
    from paper_2506_02939_b200 import pamm
    w = synth.WORKLOADS[args.workload]
    if w.dtype != "bf16":
        raise SystemExit("the fused forward pass is a bf16 tensor-core kernel")
    k = args.k or w.ks[0]
    inp = synth.make_inputs(args.workload, with_dY=False)
    b, n, m = inp.b, w.n, w.m
    X = torch.from_numpy(inp.X.view(np.int16)).view(torch.bfloat16).cuda()
    rng = np.random.default_rng([w.seed, 5])
    W = torch.from_numpy(synth.f32_to_bf16_bits(rng.standard_normal((n, m), dtype=np.float32) / np.float32(np.sqrt(n)))
                         .view(np.int16)).view(torch.bfloat16).cuda()
    dev = X.device
    Z = torch.empty((b, m), dtype=torch.bfloat16, device=dev)
    idx = torch.empty(k, dtype=torch.int32, device=dev)
    C = torch.empty((k, n), dtype=torch.bfloat16, device=dev)
    invn = torch.empty(2 * k, dtype=torch.float32, device=dev)
    f = torch.empty(b, dtype=torch.int32, device=dev)
    alpha = torch.empty(b, dtype=torch.float32, device=dev)
    sp = pamm.alloc_workspace(pamm.WS_COMPRESS, b, n, m, k, pamm.BF16, dev)
    stream = torch.cuda.current_stream()

    def fused(s):
        pamm.linear_forward(X, W, k, w.index_seed + s, Z=Z, idx_out=idx, C=C, c_invnorm=invn, f=f, alpha=alpha,
                            sort_products=sp, stream=stream)

    def product_alone(s):
        pamm.linear_forward(X, W, 0, Z=Z, stream=stream)

    def compress_alone(s):
        pamm.compress_fused(X, k, w.index_seed + s, idx_out=idx, C=C, c_invnorm=invn, f=f, alpha=alpha, sort_products=sp,
                            stream=stream)

    def torch_gemm(s):
        torch.matmul(X, W, out=Z)

    def timed(fn, steps):
        for s in range(3):
            fn(s)
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        ev[0].record(stream)
        for s in range(steps):
            fn(s)
            ev[s + 1].record(stream)
        torch.cuda.synchronize()
        return stats([ev[s].elapsed_time(ev[s + 1]) for s in range(steps)])

    K = max(5, min(args.steps, 50))
    sampler = ClockSampler(env_int("LOCAL_RANK", 0))
    sampler.start()
    launches0 = pamm.launch_count()
    t_fused = timed(fused, K)
    launches = pamm.launch_count() - launches0
    t_prod = timed(product_alone, K)
    t_comp = timed(compress_alone, K)
    t_torch = timed(torch_gemm, K)
    dX = torch.empty((b, n), dtype=torch.bfloat16, device=dev)
    t_dx = timed(lambda s: pamm.linear_backward_input(Z, W, dX=dX, stream=stream), K)     # Algorithm 3's dX = dZ W^T, dZ := Z
    t_dx_torch = timed(lambda s: torch.matmul(Z, W.t(), out=dX), K)
    clocks = sampler.stop()
    status = pamm.last_device_status()
    if status != pamm.OK:
        raise SystemExit(f"device status: {pamm.status_string(status)}")
    peak, peak_tf, peak_kind = measured_peaks()
    flops = 2.0 * b * n * (m + k)
    tf = flops / (t_fused["median"] * 1e-3) / 1e12
    line = {
        "metric": "fused forward pass Z = X W with Compress(X): tokens/s per QKV layer", "value": b / (t_fused["median"] * 1e-3),
        "unit": "tokens/s", "n_gpus": 1, "steps": K, "warmup": 3, "ms_per_step": t_fused["median"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{w.name} forward: X bf16 b={b} n={n}, W n x m={m}, k={k}", "l2": "inputs exceed L2"},
        "roofline": {"bound": "tensor", "kernel": "linear_forward_pair_kernel (X [W | C^T], 256 x 256 tiles on pairs of CTAs)", "achieved": tf,
                     "peak": peak_tf, "peak_source": f"of {peak_kind} (sustained bf16)", "unit": "TFLOP/s", "frac": tf / peak_tf,
                     "traffic": None, "algorithmic_flops": flops},
        "forward_ms": {"fused_product_and_compression": t_fused, "product_alone_same_kernel": t_prod,
                       "compression_alone": t_comp,
                       "cost_of_compression_inside_the_product_ms": t_fused["median"] - t_prod["median"],
                       "torch_matmul_context_only": t_torch,
                       "input_gradient_product_dZ_Wt": t_dx, "torch_matmul_dZ_Wt_context_only": t_dx_torch},
        "gpu_launches": int(launches), "clocks": clocks,
    }
    print(json.dumps(line), flush=True)


def run_layer_loop(args):
    """A stack of QKV layers on one GPU: every layer's forward compress keeps only (C, f, alpha),
    then the backward passes run in reverse order.  Reports tokens/s per layer and the bytes kept
    for the backward pass against storing every layer's X (the memory the method is about)."""
    import torch
    from paper_2506_02939_b200 import build as pamm_build, synth
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the PAMM path has no CPU fallback")
    torch.cuda.set_device(env_int("LOCAL_RANK", 0))
    pamm_build.build()
    from paper_2506_02939_b200 import pamm
    w = synth.WORKLOADS[args.workload]
    k = args.k or w.ks[0]
    L = args.layers
    e = 2 if w.dtype == "bf16" else 4
    dt_code = pamm.BF16 if w.dtype == "bf16" else pamm.F32
    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    D = min(L, args.distinct_layers)      # distinct input sets (seed + 100 * layer), reused cyclically

    def dev(a):
        t = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16) if a.dtype == np.uint16 else torch.from_numpy(a)
        return t.cuda()

    Xs, dYs = [], []
    for d in range(D):
        inp = synth.make_inputs(args.workload, seed=w.seed + 100 * d)
        Xs.append(dev(inp.X))
        dYs.append(dev(inp.dY))
    b, n, m = w.b, w.n, w.m
    devc = Xs[0].device
    saved = [dict(idx=torch.empty(k, dtype=torch.int32, device=devc), C=torch.empty((k, n), dtype=tdt, device=devc),
                  invn=torch.empty(2 * k, dtype=torch.float32, device=devc),
                  f=torch.empty(b, dtype=torch.int32, device=devc), alpha=torch.empty(b, dtype=torch.float32, device=devc),
                  sp=pamm.alloc_workspace(pamm.WS_COMPRESS, b, n, m, k, dt_code, devc))
             for _ in range(L)]
    dW = torch.empty((n, m), dtype=torch.float32, device=devc)
    ws = pamm.alloc_workspace(pamm.WS_CONTRACT, b, n, m, k, dt_code, devc)
    stream = torch.cuda.current_stream()

    def step(s):
        for l in range(L):
            sv = saved[l]
            pamm.compress_fused(Xs[l % D], k, w.index_seed + 100 * l + s, idx_out=sv["idx"], C=sv["C"], c_invnorm=sv["invn"],
                                f=sv["f"], alpha=sv["alpha"], sort_products=sv["sp"], stream=stream)
        for l in reversed(range(L)):
            sv = saved[l]
            pamm.contract_weight_grad(sv["C"], sv["f"], sv["alpha"], dYs[l % D], dW=dW, sort_products=sv["sp"], workspace=ws,
                                      stream=stream)

    for s in range(max(3, args.warmup)):
        step(s)
    torch.cuda.synchronize()
    K = max(1, args.steps)
    sampler = ClockSampler(env_int("LOCAL_RANK", 0))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = pamm.launch_count()
    sampler.start()
    e0.record(stream)
    for s in range(K):
        step(s)
    e1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    status = pamm.last_device_status()
    if status != pamm.OK:
        raise SystemExit(f"device status after the timed region: {pamm.status_string(status)}")
    ms = e0.elapsed_time(e1)
    kept = sum(sum(t.numel() * t.element_size() for key, t in sv.items() if key in ("C", "f", "alpha", "sp")) for sv in saved)
    full = L * b * n * e
    line = {
        "metric": METRIC, "value": b * L * K / (ms * 1e-3), "unit": "tokens/s", "n_gpus": 1, "steps": K,
        "warmup": max(3, args.warmup), "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": f"{w.name} x {L} layers: X {w.dtype} b={b} n={n}, dY b x m={m}, k={k}; forward of all layers, "
                               f"then backward in reverse; {D} distinct input sets (seed + 100 * layer) reused cyclically",
                   "l2": "inputs exceed L2"},
        "memory_saved": {"layers": L, "kept_bytes_all_layers": int(kept), "x_bytes_all_layers": int(full), "ratio": full / kept,
                         "scalars_kept": L * (k * n + 2 * b), "scalars_x": L * b * n},
        "gpu_launches": int(pamm.launch_count() - launches0), "clocks": clocks,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="timed steps (default 3000; 20 for --impl reference)")
    ap.add_argument("--warmup", type=int, default=None, help="untimed steps (default 20; 2 for --impl reference)")
    ap.add_argument("--impl", choices=["cuda", "reference"], default="cuda")
    ap.add_argument("--workload", default="c4", help="c1..c5; c4 (LLaMA-1B-shaped) is the headline configuration")
    ap.add_argument("--k", type=int, default=0, help="override the workload's generator count")
    ap.add_argument("--ref-tokens", type=int, default=16384, help="tokens per oracle pass (bounded sample)")
    ap.add_argument("--ref-budget-s", type=float, default=120.0, help="time budget of the whole --impl reference run")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--eps", type=float, default=None,
                    help="time the neighbourhood-condition path (Eq. 2, beta) with this epsilon instead of epsilon = infinity")
    ap.add_argument("--forward", action="store_true",
                    help="time the layer's forward pass with the compression fused into the product (Algorithm 2) instead")
    ap.add_argument("--dw-dtype", choices=["f32", "bf16"], default="f32", help="storage type of the weight gradient")
    ap.add_argument("--layout", choices=["nm", "mn"], default="nm", help="dW as n x m (the paper's) or m x n (out x in)")
    ap.add_argument("--layers", type=int, default=1,
                    help="with L > 1: a stack of L layers (forward of all, then backward in reverse) and its saved-activation bytes")
    ap.add_argument("--distinct-layers", type=int, default=4, help="distinct synthetic input sets in the --layers mode")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 3000 if args.impl == "cuda" else 20
    if args.warmup is None:
        args.warmup = 20 if args.impl == "cuda" else 2
    if args.impl == "cuda":
        args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    elif args.forward:
        run_forward(args)
    elif args.layers > 1:
        run_layer_loop(args)
    else:
        run_cuda(args)
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
