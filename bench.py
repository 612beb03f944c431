#!/usr/bin/env python
"""Benchmark of the EGGROLL hot path on B200.

One "step" is one pass of the whole hot path over one population batch of the 4096x4096 bf16 layer
(one token per member): perturbed forward -> centred-rank fitness shaping -> EGGROLL update.
Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "perturbed-forward population tokens/s/GPU and % of unperturbed inference"
UNIT = "population tokens/s"

# headline workload: the largest point of the 4096^2 sweep that the paper-shaped metric is quoted on
D, N_MEMBERS, RANK, SIGMA, ALPHA, SEED = 4096, 65536, 1, 0.01, 0.01, 0
# DRAM bytes of one forward launch from the profiler capture at N = 32768 (970 MB read, 252 MB written): the part that
# does not scale with N (W) and the part that does (X read twice, Y written, re-reads of X tiles), per 16384 members
FWD_TRAFFIC_W, FWD_TRAFFIC_PER_16K = 34.0e6, 594.0e6


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="egr", choices=["egr", "reference"])
    ap.add_argument("--members", type=int, default=N_MEMBERS)
    ap.add_argument("--rank", type=int, default=RANK)
    ap.add_argument("--mode", default="replicas", choices=["replicas", "sharded"],
                    help="N>1: independent replicas (default), or one population sharded over the ranks with a "
                         "fitness all-gather and the full update on every rank")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="target CPU time of the oracle sample")
    return ap.parse_args()


# ----------------------------------------------------------------------------------------------------------
def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(bf16_sustained=p.get("bf16_tflops_sustained"), bf16_burst=p.get("bf16_tflops"),
                    hbm=p.get("hbm_gbs"), source="measured")
    return dict(bf16_sustained=1400.0, bf16_burst=1590.0, hbm=6650.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons while the timed region runs (read-only queries: NVML every few
    milliseconds when the binding is there, else nvidia-smi every 100 ms).  Nothing is ever set."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int, uuid: str | None = None):
        self.index = index
        self.uuid = uuid
        self.samples = []            # (sm_mhz, max_mhz, [4 booleans])
        self.source = "nvidia-smi"
        self.stop = threading.Event()
        self.t = threading.Thread(target=self.run, daemon=True)

    def _nvml_handle(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            if self.uuid:
                u = self.uuid if self.uuid.startswith("GPU-") else "GPU-" + self.uuid
                try:
                    return pynvml, pynvml.nvmlDeviceGetHandleByUUID(u.encode())
                except Exception:
                    pass
            return pynvml, pynvml.nvmlDeviceGetHandleByIndex(self.index)
        except Exception:
            return None, None

    def run(self):
        nv, h = self._nvml_handle()
        if h is not None:
            try:
                mx = float(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))
                bits = [getattr(nv, n, 0) for n in ("nvmlClocksEventReasonHwSlowdown", "nvmlClocksEventReasonHwThermalSlowdown",
                                                     "nvmlClocksEventReasonSwThermalSlowdown", "nvmlClocksEventReasonSwPowerCap")]
                if not all(bits):
                    bits = [0x8, 0x40, 0x20, 0x4]
                get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons
                self.source = "nvml"
                while not self.stop.is_set():
                    mhz = float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                    r = int(get_reasons(h))
                    self.samples.append((mhz, mx, [bool(r & b) for b in bits]))
                    self.stop.wait(0.004)
                return
            except Exception:
                self.source = "nvidia-smi"
        while not self.stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5).stdout
                parts = [x.strip() for x in out.strip().split(",")]
                if len(parts) >= 6:
                    self.samples.append((float(parts[0]), float(parts[1]), [x.lower().startswith("active") for x in parts[2:6]]))
            except Exception:
                pass
            self.stop.wait(0.1)

    def __enter__(self):
        self.t.start()
        return self

    def __exit__(self, *a):
        self.stop.set()
        self.t.join(timeout=6)

    def mark(self):
        """Number of samples taken so far (to slice the samples of one region afterwards)."""
        return len(self.samples)

    def summary(self, lo=0, hi=None):
        smp = self.samples[lo:hi]
        if not smp:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"], "samples": 0, "source": self.source}
        sm = sorted(s[0] for s in smp)
        reasons = [n for i, n in enumerate(self.NAMES) if any(s[2][i] for s in smp)]
        return {"sm_mhz": sm[len(sm) // 2], "sm_min_mhz": sm[0], "sm_max_mhz": smp[0][1], "reasons": reasons,
                "samples": len(sm), "source": self.source}


# ----------------------------------------------------------------------------------------------------------
def oracle_sample_rate(N, r, seconds, seed=SEED):
    """Times the CPU oracle, as it stands, on a sample of S members of the same workload: explicit perturbed
    forward of those members, centred ranks of their fitness, and their rank-r terms of the update over the
    whole matrix.  Returns (tokens_per_s, S, cores, elapsed)."""
    import numpy as np

    import oracle
    import workloads
    oracle.build()
    cores = oracle.threads()
    W = workloads.linear_layer(seed, D, D, 1, bf16=True)[0]
    g = workloads.rng(seed, 1)

    def run(S):
        X = workloads.round_to_bf16(g.standard_normal((S, D)).astype(np.float32))
        t0 = time.perf_counter()
        Y = oracle.perturbed_linear(X, W, np.arange(S), 1, r, 0, seed, 0, SIGMA)
        raw = -np.sum(Y * Y, axis=1)
        shaped = oracle.fitness_shape(raw, oracle.SHAPE_CENTERED_RANK)
        oracle.es_update_block(shaped, r, 0, seed, 0, ALPHA, 0, D, 0, D)
        return time.perf_counter() - t0

    S = cores
    t = run(S)
    if t < seconds / 3:
        S = max(cores, int(S * (seconds / max(t, 1e-3)) / cores) * cores)
        S = min(S, N)
        t = run(S)
    return S / t, S, cores, t


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    per_step = max(1.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    vals = []
    S = cores = 0
    for i in range(args.warmup + args.steps):
        v, S, cores, el = oracle_sample_rate(args.members, args.rank, per_step)
        if i >= args.warmup:
            vals.append((v, el))
    value = sum(v for v, _ in vals) / len(vals)
    sample = f"{S} of {args.members} members per step: explicit forward, centred ranks, their update terms over 4096x4096"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sum(e for _, e in vals) / len(vals), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"c5_linear_4096x4096_bf16_N{args.members}_r{args.rank}_T1", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------------------
def reduce_max_ms(ms: float, device=None) -> float:
    """Max over ranks of a per-rank duration (the job is as slow as its slowest replica)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank: int, world: int, ms_per_step: float) -> float:
    """Replicas: every rank processes units_per_rank per step; value = all units / slowest rank's time."""
    return units_per_rank * world / (ms_per_step * 1e-3)


def run_egr(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    import paper_2511_16652_b200 as egr
    import workloads

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    egr.load_library()

    N, r = args.members, args.rank
    dev = torch.device("cuda", local)
    # replicas: every rank owns an independent population of N members of the same layer (no data-path collective)
    w_seed = SEED if args.mode == "sharded" else SEED + rank      # a sharded population shares one set of weights
    W32 = torch.from_numpy(workloads.linear_layer(w_seed, D, D, 1, bf16=True)[0])
    gen = torch.Generator().manual_seed(1234 + rank)
    X_host = torch.randn((N, D), generator=gen, dtype=torch.float32).to(torch.bfloat16).pin_memory()
    raw_host = torch.randn((N,), generator=gen, dtype=torch.float32).pin_memory()
    shaped_host = torch.empty((N * world if args.mode == "sharded" else N,), dtype=torch.float32).pin_memory()

    Wm = W32.to(dev)
    Wsh = Wm.to(torch.bfloat16)
    X = X_host.to(dev)
    raw = raw_host.to(dev)
    Y = torch.empty((N, D), dtype=torch.bfloat16, device=dev)
    shaped = torch.empty((N,), dtype=torch.float32, device=dev)
    ws = egr.Workspace(dev)
    ws_b = egr.Workspace(dev)

    torch.matmul(X, Wsh.t(), out=Y)              # the library's first call (handles, kernel selection) stays out of every timing
    torch.cuda.synchronize()

    sharded = args.mode == "sharded" and world > 1
    N_global = N * world if sharded else N
    if sharded:
        from paper_2511_16652_b200 import sharding
        shaped = torch.empty((N_global,), dtype=torch.float32, device=dev)

    def layer(step, flags=0):
        return egr.Layer(D, D, N, 1, r, layer_id=0, seed=SEED + step, flags=flags,
                         x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.BF16, member_base=rank * N if sharded else 0)

    fwd_marks, upd_marks = [], []                # (start, end) events round the forward / the update of every timed step

    def compute(i, Xs, raws, after_inputs_read=None, mark=False):
        L = layer(i)
        if mark:
            m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            m0.record()
        egr.egr_perturbed_linear(L, Xs, Wsh, SIGMA, Y, ws)
        if mark:
            m1.record()
            fwd_marks.append((m0, m1))
        if sharded:
            # one exchange step: N scalars per rank; afterwards every rank applies the identical full update
            full = sharding.all_gather_fitness(raws, N_global)
            egr.egr_fitness_shape(full, egr.SHAPE_CENTERED_RANK, shaped, ws_b)
            Lu = egr.Layer(D, D, N_global, 1, r, layer_id=0, seed=SEED + i, x_dtype=egr.BF16, w_dtype=egr.BF16,
                           y_dtype=egr.BF16)
        else:
            egr.egr_fitness_shape(raws, egr.SHAPE_CENTERED_RANK, shaped, ws_b)
            Lu = L
        if after_inputs_read is not None:
            after_inputs_read()
        if mark:
            u0, u1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            u0.record()
        egr.egr_es_update(Lu, Wm, shaped, ALPHA, ws, W_shadow=Wsh)
        if mark:
            u1.record()
            upd_marks.append((u0, u1))

    def step_device(i):
        compute(i, X, raw, mark=(i >= args.warmup))      # the dominant kernel is timed live, inside the timed region

    # End to end: every step copies that step's inputs from pinned host memory and reads the shaped fitness back.
    # The copy of step i+1's inputs runs on a copy stream into the other of two device buffers while step i
    # computes, so the steady-state step costs max(copy, compute); every step still pays its own copy.
    copy_stream = torch.cuda.Stream(device=dev)
    X_buf = [X, torch.empty_like(X)]
    raw_buf = [raw, torch.empty_like(raw)]
    copied = [torch.cuda.Event(), torch.cuda.Event()]
    consumed = [torch.cuda.Event(), torch.cuda.Event()]
    e2e_state = {"primed": False, "n": 0}

    def enqueue_copy(slot):
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(consumed[slot])          # the buffer's previous contents have been used
            X_buf[slot].copy_(X_host, non_blocking=True)
            raw_buf[slot].copy_(raw_host, non_blocking=True)
            copied[slot].record(copy_stream)

    def step_e2e(i):
        main = torch.cuda.current_stream()
        n = e2e_state["n"]
        slot = n & 1
        if not e2e_state["primed"]:
            consumed[0].record(main); consumed[1].record(main)
            enqueue_copy(slot)
            e2e_state["primed"] = True
        enqueue_copy(slot ^ 1)                               # next step's inputs, overlapping this step's compute
        main.wait_event(copied[slot])
        compute(i, X_buf[slot], raw_buf[slot], after_inputs_read=lambda: consumed[slot].record(main))
        shaped_host.copy_(shaped, non_blocking=True)
        e2e_state["n"] = n + 1

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, warmup, base=0, sampler=None):
        for i in range(warmup):
            fn(base + i)
        barrier()
        lo = sampler.mark() if sampler is not None else 0
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            fn(base + warmup + i)
        e1.record()
        barrier()
        if sampler is not None:
            timed.span = (lo, sampler.mark())
        return reduce_max_ms(e0.elapsed_time(e1), dev) / steps

    def time_call(fn, reps=10, warm=3):
        """Average device time of one call (CUDA events on the launching stream)."""
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    uuid = str(getattr(torch.cuda.get_device_properties(local), "uuid", "")) or None
    with ClockSampler(local, uuid) as clocks:
        ms_step = timed(step_device, args.steps, args.warmup, sampler=clocks)
        # The library GEMM in the regime the steps just ran in: a loop of about the same length, started right behind
        # them without a pause, so that it sees the clocks (burst or power-capped) that the timed forward saw.
        n_lib = max(3, int(args.steps * ms_step / 1.4))
        lib0, lib1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        lib0.record()
        for _ in range(n_lib):
            torch.matmul(X, Wsh.t(), out=Y)
        lib1.record()
        torch.cuda.synchronize()
        ms_torch_regime = lib0.elapsed_time(lib1) / n_lib
    clk = clocks.summary(*timed.span)
    status = egr.egr_workspace_status(ws)
    if status != 0:
        raise SystemExit(f"device-side status: {egr.egr_strerror(status)}")
    ms_e2e = timed(step_e2e, max(2, args.steps // 2), 1, base=1000)

    # components (device time per call, same buffers; inputs exceed L2 so no flush is needed)
    L0 = layer(5000)
    ms_fwd = time_call(lambda: egr.egr_perturbed_linear(L0, X, Wsh, SIGMA, Y, ws))
    Lp = layer(5000, egr.NO_PERTURB)
    ms_plain = time_call(lambda: egr.egr_perturbed_linear(Lp, X, Wsh, SIGMA, Y, ws))
    ms_torch = time_call(lambda: torch.matmul(X, Wsh.t(), out=Y))
    ms_shape = time_call(lambda: egr.egr_fitness_shape(raw, egr.SHAPE_CENTERED_RANK, shaped, ws_b))
    ms_upd = time_call(lambda: egr.egr_es_update(L0, Wm, shaped, ALPHA, ws, W_shadow=Wsh), reps=5, warm=2)

    # memory-bound pieces: achieved algorithmic GB/s (8 bytes per member: one read, one write) against the measured copy
    # bandwidth.  At the bench's N they move 512 KB and are bound by launch latency; a population of 2^25 members
    # (268 MB, larger than L2) shows what the same kernels reach when bandwidth is the limit.
    pk = peaks()
    raw_eq = torch.full_like(raw, -2650.25)
    raw_band = (-2650.0 + 2.0 * torch.rand(N, device=dev) - 1.0).contiguous()
    ms_shape_eq = time_call(lambda: egr.egr_fitness_shape(raw_eq, egr.SHAPE_CENTERED_RANK, shaped[:N], ws_b))
    ms_shape_band = time_call(lambda: egr.egr_fitness_shape(raw_band, egr.SHAPE_CENTERED_RANK, shaped[:N], ws_b))
    NB = 1 << 25
    big_raw = torch.randn(NB, device=dev)
    big_out = torch.empty(NB, device=dev)
    membound = []
    # moved = bytes the kernels actually read and write per member: z-score reads the values three times (sum, squared
    # deviations, apply) and writes once
    for name, mode, n_, src, dst, moved in (("zscore (zs_sum, zs_var, zs_apply)", egr.SHAPE_ZSCORE, NB, big_raw, big_out, 16),
                                            ("pair_sign", egr.SHAPE_ANTITHETIC_SIGN, NB, big_raw, big_out, 8),
                                            ("zscore (zs_sum, zs_var, zs_apply)", egr.SHAPE_ZSCORE, N, raw, shaped[:N], 16),
                                            ("pair_sign", egr.SHAPE_ANTITHETIC_SIGN, N, raw, shaped[:N], 8),
                                            ("centred_rank (radix sort of key/index pairs)", egr.SHAPE_CENTERED_RANK, N, raw, shaped[:N], 68)):
        ms = time_call(lambda: egr.egr_fitness_shape(src, mode, dst, ws_b))
        gbs = 8.0 * n_ / (ms * 1e-3) / 1e9
        membound.append({"kernel": name, "members": n_, "ms": ms, "algorithmic_bytes": 8 * n_, "gbs": gbs,
                         "frac_of_measured_hbm": gbs / pk["hbm"], "moved_bytes": moved * n_,
                         "moved_gbs": moved * n_ / (ms * 1e-3) / 1e9, "moved_frac_of_measured_hbm": moved * n_ / (ms * 1e-3) / 1e9 / pk["hbm"]})
    del big_raw, big_out

    flops_fwd = 2.0 * N * D * D
    # the forward's launch (a workspace memset of a few KB and the kernel) as it ran inside the timed steps
    ms_fwd_in_step = sum(a.elapsed_time(b) for a, b in fwd_marks) / max(1, len(fwd_marks))
    achieved = flops_fwd / (ms_fwd_in_step * 1e-3) / 1e12
    ms_upd_in_step = sum(a.elapsed_time(b) for a, b in upd_marks) / max(1, len(upd_marks))
    K = N_global * r
    upd_tflops_in_step = 2.0 * D * D * K / (ms_upd_in_step * 1e-3) / 1e12
    lib_tflops_regime = flops_fwd / (ms_torch_regime * 1e-3) / 1e12
    # Which measured peak is the denominator: MEASURED_PEAKS has a burst figure (a GEMM timed alone for milliseconds, at
    # boost clocks) and a sustained one (seconds under the power cap).  The clocks sampled during the timed region say
    # which of the two it ran in; and whatever they say, a peak that the library GEMM beats in this very run, in the
    # same regime, is not the peak of that regime.
    region_s = ms_step * args.steps * 1e-3
    have_clk = clk.get("sm_mhz") is not None and bool(clk.get("sm_max_mhz"))
    near_max = have_clk and clk["sm_mhz"] >= 0.92 * clk["sm_max_mhz"]
    capped = have_clk and not near_max and "sw_power_cap" in clk.get("reasons", [])
    if have_clk:
        # the sampled clocks decide: a region that ran under the power cap with its median clock well below the maximum
        # is the sustained regime however short it was, one that held the boost clock is the burst regime however long
        regime = "sustained" if capped else "burst"
        why = "timed region %.2f s, median SM clock %.0f of %.0f MHz%s" % (
            region_s, clk["sm_mhz"], clk["sm_max_mhz"], ", power cap active" if capped else "")
    else:
        regime = "burst" if region_s < 1.0 else "sustained"
        why = "timed region %.2f s, no clock samples" % region_s
    if regime == "sustained" and lib_tflops_regime > 1.02 * pk["bf16_sustained"]:
        regime, why = "burst", why + ", library GEMM in the same regime exceeds the sustained figure"
    peak = pk["bf16_burst"] if regime == "burst" else pk["bf16_sustained"]
    nominal = 2250.0
    chunks = -(-K // 8192)                       # update K-chunk for a 4096x4096 layer
    # kernels per step: the fused forward; the radix-sort ranks (1 + 4 x 2); the update - for ranks below 4 and K >= 8192
    # one launch that stages and contracts plus the bf16 shadow pass, otherwise two staging kernels and one GEMM per chunk
    one_launch = r < 4 and (chunks >= 4 or K >= 8192)        # the library's rule for a 4096 x 4096 layer
    launches_per_step = 1 + 9 + (2 if one_launch else 3 * chunks)
    tokens = N * world
    pct_own, pct_torch = 100.0 * ms_plain / ms_fwd, 100.0 * ms_torch / ms_fwd
    pct_torch_regime = 100.0 * ms_torch_regime / ms_fwd_in_step

    line = {
        "metric": METRIC, "value": whole_job_value(N, world, ms_step), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"c5_linear_4096x4096_bf16_N{N}_r{r}_T1", "step": "forward+centred_rank+update",
                   "members_per_gpu": N, "rank": r, "sigma": SIGMA, "alpha": ALPHA, "l2": "inputs_exceed_l2",
                   "parallelism": (f"population_sharded{world}" if sharded else f"replicas{world}")},
        "forward": {"tokens_per_s": N / (ms_fwd * 1e-3), "ms": ms_fwd, "ms_in_step": ms_fwd_in_step, "ms_unperturbed_own": ms_plain,
                    "ms_unperturbed_torch": ms_torch, "ms_unperturbed_torch_in_regime": ms_torch_regime,
                    "pct_of_unperturbed_own": pct_own, "pct_of_unperturbed_torch": pct_torch,
                    "pct_of_unperturbed_torch_in_regime": pct_torch_regime},
        "shape": {"ms": ms_shape, "ms_all_equal": ms_shape_eq, "ms_narrow_band": ms_shape_band,
                  "gbs": 8.0 * N / (ms_shape * 1e-3) / 1e9},
        "memory_bound": membound,
        "update": {"ms": ms_upd, "ms_in_step": ms_upd_in_step, "tflops": 2.0 * D * D * K / (ms_upd * 1e-3) / 1e12,
                   "tflops_in_step": upd_tflops_in_step, "frac_of_peak_in_step": upd_tflops_in_step / peak,
                   "w_gbs": (D * D * (4 + 4 + 2)) / (ms_upd * 1e-3) / 1e9,
                   # one fp32 read and write of W per K-chunk, the bf16 shadow once, the fitness
                   "algorithmic_bytes": D * D * 8 * chunks + D * D * 2 + 4 * N_global,
                   "gbs": (D * D * 8 * chunks + D * D * 2 + 4 * N_global) / (ms_upd * 1e-3) / 1e9},
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                     "frac": achieved / peak, "regime": regime, "regime_why": why,
                     "frac_burst": achieved / pk["bf16_burst"], "frac_sustained": achieved / pk["bf16_sustained"],
                     "peak_nominal": nominal, "frac_nominal": achieved / nominal,
                     "ms_times_median_sm_mhz": (ms_fwd_in_step * clk["sm_mhz"]) if clk.get("sm_mhz") else None,
                     "library_gemm_same_regime": {"tflops": lib_tflops_regime, "frac": lib_tflops_regime / peak},
                     # dram bytes of one launch: captured at N = 16384 and scaled with N (all but the 34 MB of W scale)
                     "traffic": FWD_TRAFFIC_W + FWD_TRAFFIC_PER_16K * (N / 16384.0), "peak_source": pk["source"],
                     "algorithmic_bytes": N * D * 2 + D * D * 2 + N * D * 2,
                     "kernel": "gemm_sm100_kernel<FORWARD> (tcgen05 CTA-pair GEMM, side-warp skinny products, fused rank-r epilogue)",
                     "timed": "CUDA events round the forward call of every timed step (forward.ms_in_step); forward.ms is the same call timed alone",
                     "traffic_note": "ncu capture at N=32768 scaled to this N, see profiles/forward_gemm_c5_N32768_r1.md"},
        "targets": {
            "forward_pct_of_unperturbed_ge_85": {"value": min(pct_own, pct_torch), "met": bool(min(pct_own, pct_torch) >= 85.0),
                                                 "note": "the stricter of own unperturbed kernel and torch.matmul, each timed alone"},
            "forward_frac_of_nominal_dense_bf16_ge_0.60": {"value": achieved / nominal, "met": bool(achieved / nominal >= 0.60)},
            "forward_frac_of_measured_peak_ge_0.60": {"value": achieved / peak, "met": bool(achieved / peak >= 0.60)},
        },
        "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": N * D * 2 + N * 4,
                "d2h_bytes_per_step": N * 4, "ms_per_step": ms_e2e,
                "note": "inputs copied from pinned host memory every step (double-buffered, overlapped with compute)"},
        "gpu_launches": launches_per_step * args.steps,
        "clocks": clk,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, S, cores, el = oracle_sample_rate(N, r, args.cpu_seconds)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"{S} of {N} members: explicit forward, centred ranks, their update terms "
                                          f"over 4096x4096 ({el:.1f} s)"}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    a = parse()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_egr(a)
