"""Benchmark of the RDK hot path on B200.

One "step" takes one batch of the Llama-3-scale workload C2 (target vocabulary N = 128256, drafter
keeps n = 32064 ids, 64 sequences x 5 draft positions = 320 rows, bf16 logits) through the whole
path: drafter/target soft-max, Token-Level Intersection, first-order redistribution, draft draw,
rejection test, acceptance rate, residual draw and the per-sequence accepted length.  The metric
is verified draft tokens per second = rows x steps / elapsed.  The same line carries, under
"workloads", the other sizes of the linear path (C3, C4) against the HBM roofline and the exact
tensor-core path (C5) against the bf16 tensor peak.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload C2|C3|C4|C5]

Prints ONE JSON line.  With --impl reference the CPU checker (oracle/) is timed on the host cores
instead; that arm touches no GPU.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOAD = "C2"              # the configuration the metric is quoted on (--workload picks another as the headline)
OTHER_WORKLOADS = ("C3", "C4", "C5", "T1")
N_BUFFER_SETS = 6            # distinct input batches rotated through, so every step reads HBM
METRIC = "verified draft tokens/sec"
UNIT = "tokens/s"
MIN_TIMED_SECONDS = 0.5      # the K-step loop is repeated until at least this much has been timed (and 5 times)

# DRAM traffic of one launch of the dominant kernel from an ncu capture
# (dram__bytes_read.sum + dram__bytes_write.sum), valid only for the kernel sources with this hash.
NCU_TRAFFIC = {"sources_sha256": "1e0aa2b1d5ccce991f824bee5f0645738ce82e870d36d720dafa90eb37320f60",
               "bytes_per_launch": {"C2": 106771456, "C3": 586242560}}
KERNEL_SOURCES = ("rdk_row_stream.cu", "rdk_row.cuh", "rdk_common.cuh")


def _kernel_sources_hash() -> str:
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2506_03206_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def _measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm": float(d["hbm_gbs"]), "tensor": float(d["bf16_tflops"]), "tensor_sustained": float(d["bf16_tflops_sustained"]),
                "source": "measured (MEASURED_PEAKS.json: hbm_gbs, bf16_tflops burst, bf16_tflops_sustained)"}
    return {"hbm": 6650.0, "tensor": 1590.0, "tensor_sustained": 1400.0,
            "source": "fallback (6.65 TB/s, 1.59 / 1.4 PFLOP/s: earlier measurements on this pool)"}


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons of one GPU through NVML while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, torch_device_index: int, period_s: float = 0.01):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = str(torch.cuda.get_device_properties(torch_device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(torch_device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as e:  # NVML missing: the bench still runs, the clocks entry says so
            self.err = repr(e)

    def _reasons(self) -> int:
        nv = self.nv
        for fn in ("nvmlDeviceGetCurrentClocksEventReasons", "nvmlDeviceGetCurrentClocksThrottleReasons"):
            if hasattr(nv, fn):
                try:
                    return int(getattr(nv, fn)(self.h))
                except Exception:
                    continue
        return 0

    def run(self):
        if not self.ok:
            return
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                bits = self._reasons()
                for b, name in self.REASONS.items():
                    if bits & b:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=1.0)

    def summary(self):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["nvml unavailable"]}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


# ----------------------------------------------------------------------------------------------
# the CPU checker as a timed baseline (the one place besides --impl reference where oracle/ runs)
# ----------------------------------------------------------------------------------------------
def _cpu_baseline_linear(cfg, name: str, min_seconds: float = 10.0, pool_rows: int = 64):
    """Time the CPU checker, as it stands, on rows of the same workload for about min_seconds."""
    import numpy as np

    import workloads as W
    from oracle import rdk_oracle as O
    inp = W.make_inputs(cfg.with_rows(pool_rows, 1), device="cpu")
    kappa = inp["kept_ids"].numpy()
    z = [W.to_f64(inp["target"][r]) for r in range(pool_rows)]
    y = [W.to_f64(inp["drafter"][r]) for r in range(pool_rows)]
    u = inp["uniforms"].numpy().astype(np.float64)
    done = 0
    t0 = time.perf_counter()
    while True:
        r = done % pool_rows
        O.rdk_row(z[r], y[r], kappa, u[r], "linear", drafter_kind=cfg.drafter_kind)
        done += 1
        dt = time.perf_counter() - t0
        if dt >= min_seconds:
            break
    return {"value": done / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{done} rows of {name} through oracle.rdk_row (float64 numpy, one thread, {dt:.1f} s)"}


def _cpu_baseline_exact(cfg, name: str, rows: int = 256, cols: int = 4096):
    """The checker's exact path on a bounded sample: `rows` rows, the contraction on `cols` seeded columns of
    the affinity matrix (built by the checker beforehand, untimed like the library's preprocessing) and scaled to
    all N columns, plus the checker's sampling step on a weight vector of full length."""
    import numpy as np

    import workloads as W
    from oracle import rdk_oracle as O
    inp = W.make_inputs(cfg.with_rows(rows, 1), device="cpu", with_embeddings=True)
    kappa = inp["kept_ids"].numpy()
    rng = np.random.default_rng(cfg.seed)
    sel = np.sort(rng.choice(cfg.N, cols, replace=False))
    Mcols = O.round_to_bf16(O.affinity_columns(W.to_f64(inp["embeddings"]), kappa, cfg.tau, sel))
    z = [W.to_f64(inp["target"][r]) for r in range(rows)]
    y = [W.to_f64(inp["drafter"][r]) for r in range(rows)]
    u = inp["uniforms"].numpy().astype(np.float64)
    t0 = time.perf_counter()
    wc = []
    for r in range(rows):
        qk = O.round_to_bf16(O.drafter_qprime(y[r], kappa, cfg.N, cfg.drafter_kind)[kappa])
        wc.append(O.redistribute_exact(qk, Mcols))
    t_contract = (time.perf_counter() - t0) * (cfg.N / cols)
    t0 = time.perf_counter()
    for r in range(rows):
        O.rdk_row(z[r], None, kappa, u[r], "given", w_given=np.resize(wc[r], cfg.N))
    t_sample = time.perf_counter() - t0
    dt = t_contract + t_sample
    return {"value": rows / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": (f"{rows} rows of {name}: oracle.redistribute_exact on {cols} of {cfg.N} seeded columns of the checker's "
                       f"bf16-rounded affinity matrix, time scaled by {cfg.N / cols:.1f} ({t_contract:.1f} s), plus oracle.rdk_row "
                       f"(mode 'given') on full-length weights ({t_sample:.1f} s); float64 numpy, one thread")}


def run_reference(args):
    """--impl reference: the CPU checker timed on the host cores; rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np

    import workloads as W
    from oracle import rdk_oracle as O
    cfg = W.CONFIGS[args.workload]
    if cfg.path == "exact":
        raise SystemExit("--impl reference times the benchmark's linear workloads only")
    total_steps = args.steps + args.warmup
    per_row_s = 0.04
    rows_per_step = int(max(1, min(64, cfg.rows, 120.0 / (per_row_s * max(1, total_steps)))))
    pool = min(cfg.rows, max(rows_per_step, 16))
    inp = W.make_inputs(cfg.with_rows(pool, 1), device="cpu")
    kappa = inp["kept_ids"].numpy()
    z = [W.to_f64(inp["target"][r]) for r in range(pool)]
    y = [W.to_f64(inp["drafter"][r]) for r in range(pool)]
    u = inp["uniforms"].numpy().astype(np.float64)

    def step(i):
        for k in range(rows_per_step):
            r = (i * rows_per_step + k) % pool
            O.rdk_row(z[r], y[r], kappa, u[r], "linear", drafter_kind=cfg.drafter_kind)

    for i in range(args.warmup):
        step(i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        step(args.warmup + i)
    dt = time.perf_counter() - t0
    value = rows_per_step * args.steps / dt
    sample = f"{rows_per_step} row(s) of {args.workload} per step through oracle.rdk_row (float64 numpy, one thread)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{args.workload}: N={cfg.N} n={cfg.n} bf16 logits, linear RDK; {sample}"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def max_over_ranks(ms: float, dist, device) -> float:
    """Slowest rank's time: the job is as fast as its slowest replica."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(rows_per_rank: int, trials: int, steps: int, world: int, ms: float) -> float:
    """Units all ranks processed divided by the slowest rank's time (replicas: weak scaling)."""
    return world * rows_per_rank * trials * steps / (ms * 1e-3)


def repeats_for(est_ms_per_step: float, steps: int, min_seconds: float = MIN_TIMED_SECONDS) -> int:
    """How often the K-step loop is timed: at least five times and until min_seconds have been timed."""
    per_loop = max(est_ms_per_step * steps * 1e-3, 1e-6)
    return int(min(2000, max(5, math.ceil(min_seconds / per_loop))))


def median_and_spread(xs):
    s = sorted(xs)
    med = s[len(s) // 2] if len(s) % 2 else 0.5 * (s[len(s) // 2 - 1] + s[len(s) // 2])
    return med, (s[-1] - s[0]) / med if med > 0 else 0.0


class Ctx:
    def __init__(self, torch, B, W, dist, dev, world, rank, local_rank, peaks):
        self.torch, self.B, self.W, self.dist, self.dev = torch, B, W, dist, dev
        self.world, self.rank, self.local_rank, self.peaks = world, rank, local_rank, peaks

    def barrier(self):
        self.torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
            self.torch.cuda.synchronize()

    def timed(self, fn, n_steps: int) -> float:
        """Exactly n_steps steps between two events, a barrier and a synchronise on both sides; max over ranks."""
        t = self.torch
        e0, e1 = t.cuda.Event(enable_timing=True), t.cuda.Event(enable_timing=True)
        self.barrier()
        e0.record()
        for i in range(n_steps):
            fn(i)
        e1.record()
        self.barrier()
        return max_over_ranks(e0.elapsed_time(e1), self.dist, self.dev)

    def timed_repeats(self, fn, n_steps: int, warm_ms: float):
        reps = repeats_for(warm_ms / max(1, n_steps), n_steps)
        return [self.timed(fn, n_steps) for _ in range(reps)]


def bench_workload(ctx: Ctx, name: str, steps: int, warmup: int, prior: bool, headline: bool, cpu_baseline: bool):
    """Time one workload; returns the fields of its entry (the headline workload's become the line itself)."""
    torch, B, W, dev = ctx.torch, ctx.B, ctx.W, ctx.dev
    cfg = W.CONFIGS[name]
    exact = cfg.path == "exact"
    rows, trials = cfg.rows, cfg.trials
    zb = 2 if cfg.dtype == "bf16" else 4
    kind = B.RDK_PROBS if cfg.drafter_kind == "probs" else B.RDK_LOGITS
    row_bytes = cfg.N * zb + cfg.n * zb + trials * 16 + 30
    # enough distinct batches that one rotation exceeds L2 several times over (C5's operands do so alone)
    nsets = 1 if exact else max(2, min(N_BUFFER_SETS, int(600e6 // (rows * row_bytes)) + 1))
    sets = [W.make_inputs(cfg, device=str(dev), variant=v + 100 * ctx.rank, with_embeddings=exact and v == 0)
            for v in range(nsets)]
    index = B.rdk_prepare_ids(sets[0]["kept_ids"], cfg.N)
    outs = [B.alloc_outputs(rows, cfg.batch, trials, dev) for _ in range(nsets)]
    outs_nolen = [{k: v for k, v in o.items() if k != "accepted_len"} for o in outs]
    pb = B.make_problem(index, sets[0]["target"], sets[0]["drafter"], cfg.batch, cfg.positions, kind)
    ws = B.sample_workspace(pb, B.RDK_MODE_LINEAR, trials, dev)

    prep_ms = None
    kernels = None
    if exact:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        M = B.rdk_build_affinity(sets[0]["embeddings"], sets[0]["kept_ids"], cfg.tau, B.RDK_AFF_BF16_COLS)
        e1.record()
        torch.cuda.synchronize()
        prep_ms = e0.elapsed_time(e1)
        w_buf = torch.empty(rows, cfg.N, dtype=torch.float32, device=dev)
        _, _, ews = B.rdk_redistribute_exact(index, sets[0]["drafter"], M, cfg.batch, cfg.positions, kind, w_out=w_buf)

        def contraction(i):
            B.rdk_redistribute_exact(index, sets[0]["drafter"], M, cfg.batch, cfg.positions, kind, w_out=w_buf, ws=ews)

        def step(i, out_list=outs):
            contraction(i)
            B.rdk_sample_and_verify(index, B.RDK_MODE_PRECOMPUTED_W, sets[0]["target"], None, w_buf, sets[0]["uniforms"],
                                    cfg.batch, cfg.positions, kind, out=out_list[0], ws=ws)
        kernel_fn = contraction
        launches_per_step = 2 + 2          # operand, contraction; row kernel, accepted length
        kernels = "exact_operand_kernel + exact_tc_kernel (row sums in its epilogue)"
    elif prior:
        # Eq. rdk-taylor with one shared prior row (a static stand-in for the unknown target distribution)
        shared_prior = sets[-1]["target"][0].clone().contiguous()

        def step(i, out_list=outs):
            s = sets[i % nsets]
            B.rdk_sample_and_verify_prior(index, s["target"], shared_prior, s["drafter"], s["uniforms"],
                                          cfg.batch, cfg.positions, kind, out=out_list[i % nsets])
        kernel_fn = lambda i: step(i, outs_nolen)
        launches_per_step = 2              # row kernel, accepted length
        kernels = "rdk_row_kernel (shared prior)"
    else:
        route, why = B.rdk_sample_route(index, B.RDK_MODE_LINEAR, sets[0]["target"], sets[0]["drafter"], cfg.batch,
                                        cfg.positions, trials, ws, kind)
        if route != B.RDK_ROUTE_STREAM_KERNEL:
            raise SystemExit(f"{name}: the benchmark shape would take the one-CTA-per-row kernel ({why}); refusing to time it")

        def step(i, out_list=outs):
            s = sets[i % nsets]
            B.rdk_sample_and_verify(index, B.RDK_MODE_LINEAR, s["target"], s["drafter"], None, s["uniforms"],
                                    cfg.batch, cfg.positions, kind, out=out_list[i % nsets], ws=ws)
        kernel_fn = lambda i: step(i, outs_nolen)
        launches_per_step = 2              # stream kernel, draw kernel
        kernels = "rdk_stream_kernel + rdk_draw_kernel (route reported by rdk_sample_route)"

    for i in range(max(3, warmup)):
        step(i)
    warm_ms = ctx.timed(step, steps)                   # a first, untimed-for-the-record pass sizes the number of repeats
    sampler = ClockSampler(ctx.local_rank)
    sampler.start()
    loop_ms = ctx.timed_repeats(step, steps, warm_ms)
    # the dominant kernels alone: linear = stream + draw kernels; exact = the contraction call
    # (operand preparation, tensor-core kernel, row sums)
    kern_ms = ctx.timed_repeats(kernel_fn, steps, warm_ms)
    sampler.stop()
    B.check_status_word(outs[0], f"bench step {name}")
    burst_ms = None
    if exact:
        # The same call under the condition the burst peak was measured in: short runs (about 20 ms) that start
        # from an idle device, before the power cap pulls the clocks down; the loops above are the sustained case.
        bursts = []
        for _ in range(3):
            torch.cuda.synchronize()
            time.sleep(1.0)
            bursts.append(ctx.timed(kernel_fn, 50) / 50)
        burst_ms = sorted(bursts)[1]
    ms, spread = median_and_spread(loop_ms)
    kms, kspread = median_and_spread(kern_ms)
    kernel_ms = kms / steps

    e2e = None
    if not prior:
        e2e_steps = max(3, min(steps, 20))
        if not exact:
            # end to end: host (pinned) buffers in, host results out, copies inside the timed region
            host_sets = [{k: s[k].cpu().pin_memory() for k in ("target", "drafter", "uniforms")} for s in sets[:2]]
            stage = {"target": torch.empty_like(sets[0]["target"]), "drafter": torch.empty_like(sets[0]["drafter"]),
                     "uniforms": torch.empty_like(sets[0]["uniforms"]), "ws": ws}
            host_out = {k: torch.empty_like(v, device="cpu").pin_memory() for k, v in outs[0].items() if not k.startswith("_")}

            def e2e_step(i):
                h = host_sets[i % len(host_sets)]
                B.rdk_sample_and_verify_host(index, h["target"], h["drafter"], h["uniforms"], cfg.batch, cfg.positions,
                                             stage, outs[0], host_out, kind)
            how = "rdk_sample_and_verify_host (pinned host buffers in, host results out)"
        else:
            # the exact path has no host entry point of its own: the same two calls a user makes, with the
            # step's inputs copied in from pinned host memory and the results copied back, all inside the timed region
            host_in = {k: sets[0][k].cpu().pin_memory() for k in ("target", "drafter", "uniforms")}
            stage = {k: torch.empty_like(sets[0][k]) for k in host_in}
            host_out = {k: torch.empty_like(v, device="cpu").pin_memory() for k, v in outs[0].items() if not k.startswith("_")}

            def e2e_step(i):
                for k in stage:
                    stage[k].copy_(host_in[k], non_blocking=True)
                B.rdk_redistribute_exact(index, stage["drafter"], M, cfg.batch, cfg.positions, kind, w_out=w_buf, ws=ews)
                B.rdk_sample_and_verify(index, B.RDK_MODE_PRECOMPUTED_W, stage["target"], None, w_buf, stage["uniforms"],
                                        cfg.batch, cfg.positions, kind, out=outs[0], ws=ws)
                for k, v in host_out.items():
                    v.copy_(outs[0][k], non_blocking=True)
                torch.cuda.synchronize()
            host_sets = [host_in]
            how = "rdk_redistribute_exact + rdk_sample_and_verify between copies from and to pinned host memory"
        for i in range(3):
            e2e_step(i)
        ms_e2e = ctx.timed(e2e_step, e2e_steps)
        h2d = sum(host_sets[0][k].numel() * host_sets[0][k].element_size() for k in ("target", "drafter", "uniforms"))
        d2h = sum(v.numel() * v.element_size() for v in host_out.values())
        e2e = {"value": ctx.world * rows * trials * e2e_steps / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps, "through": how}

    peaks = ctx.peaks
    if exact:
        flops = 2.0 * rows * cfg.n * cfg.N
        achieved = flops / (kernel_ms * 1e-3) / 1e12
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peaks["tensor"], "unit": "TFLOP/s",
                    "frac": achieved / peaks["tensor"], "traffic": None, "kernel_ms": kernel_ms, "flops_per_launch": flops,
                    "peak_source": peaks["source"], "frac_of_sustained_peak": achieved / peaks["tensor_sustained"],
                    "tensor_pipe_pct_of_measured_peak": 100.0 * achieved / peaks["tensor"], "kernels": kernels,
                    "burst": {"kernel_ms": burst_ms, "achieved": flops / (burst_ms * 1e-3) / 1e12,
                              "frac_of_burst_peak": flops / (burst_ms * 1e-3) / 1e12 / peaks["tensor"],
                              "how": "median of 3 runs of 50 calls, each run after 1 s of idle"}}
    else:
        algo_bytes = rows * row_bytes
        achieved = algo_bytes / (kernel_ms * 1e-3) / 1e9
        traffic = None
        if not prior and NCU_TRAFFIC["sources_sha256"] == _kernel_sources_hash():
            traffic = NCU_TRAFFIC["bytes_per_launch"].get(name)
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm"], "unit": "GB/s", "frac": achieved / peaks["hbm"],
                    "traffic": traffic, "kernel_ms": kernel_ms, "algorithmic_bytes_per_launch": algo_bytes,
                    "peak_source": peaks["source"], "kernels": kernels}

    cpu = None
    parity = None
    if ctx.rank == 0 and cpu_baseline and not prior:
        cpu = _cpu_baseline_exact(cfg, name) if exact else _cpu_baseline_linear(cfg, name)
    if ctx.rank == 0 and not exact and not prior:
        parity = _parity_in_this_run(ctx, cfg, sets[0], outs, index, kind, ws)

    what = ("exact RDK on tensor cores (bf16 affinity, fp32 accumulate) + sampling/verification" if exact
            else "linear RDK with one shared prior row in Eq. rdk-taylor + sampling/verification" if prior
            else "linear RDK (first-order redistribution + sampling/verification)")
    entry = {
        "value": whole_job_value(rows, trials, steps, ctx.world, ms), "unit": UNIT, "ms_per_step": ms / steps,
        "timed": {"steps_per_repeat": steps, "repeats": len(loop_ms), "spread": spread, "kernel_repeats": len(kern_ms),
                  "kernel_spread": kspread, "statistic": "median over repeats of exactly `steps` steps each"},
        "config": {"workload": f"{name}: {what}, N={cfg.N}, n={cfg.n}, batch={cfg.batch}, "
                               f"positions={cfg.positions} (rows={rows}), bf16 inputs, trials={trials}",
                   "rows_per_step": rows, "parallelism": f"replicas x{ctx.world} (no collective)",
                   "l2": (f"operands of one step ({(cfg.N * cfg.n * 2 + rows * cfg.N * 4) / 1e6:.0f} MB) exceed the 126 MB L2"
                          if exact else
                          f"inputs rotate over {nsets} distinct batches ({nsets * rows * row_bytes / 1e6:.0f} MB > 126 MB L2)")},
        "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches_per_step * steps,
        "clocks": sampler.summary(), "parity": parity,
    }
    if prep_ms is not None:
        entry["config"]["preprocessing_ms"] = prep_ms
    del sets, outs, outs_nolen, ws
    torch.cuda.empty_cache()
    return entry


def _parity_in_this_run(ctx: Ctx, cfg, s0, outs, index, kind, ws, nrows: int = 16):
    """Rows of this very run recomputed by the CPU checker: how many agree, and how many draws sit on a CDF
    boundary (counted, not failed).  A handful of rows: the test-suite does the thorough comparison."""
    import numpy as np

    from oracle import rdk_oracle as O
    torch, B, W = ctx.torch, ctx.B, ctx.W
    out = outs[0]
    B.rdk_sample_and_verify(index, B.RDK_MODE_LINEAR, s0["target"], s0["drafter"], None, s0["uniforms"], cfg.batch, cfg.positions,
                            kind, out=out, ws=ws)
    torch.cuda.synchronize()
    rng = np.random.default_rng(0)
    rows = sorted(rng.choice(cfg.rows, min(nrows, cfg.rows), replace=False).tolist())
    kappa = s0["kept_ids"].cpu().numpy()
    res = {"rows_compared": len(rows), "max_abs_alpha": 0.0, "max_abs_theta": 0.0, "draft_equal": 0, "out_token_equal": 0,
           "ambiguous_draft": 0, "ambiguous_accept": 0, "ambiguous_residual": 0, "mismatches": 0}
    d, o, acc = (out[k].cpu().numpy() for k in ("draft_token", "out_token", "accepted"))
    tol = 1e-5
    for r in rows:
        u = s0["uniforms"][r].cpu().numpy().astype(np.float64)
        ref = O.rdk_row(W.to_f64(s0["target"][r]), W.to_f64(s0["drafter"][r]), kappa, u, "linear", drafter_kind=cfg.drafter_kind)
        res["max_abs_alpha"] = max(res["max_abs_alpha"], abs(float(out["alpha"][r]) - ref["alpha"]))
        res["max_abs_theta"] = max(res["max_abs_theta"], abs(float(out["theta"][r]) - ref["theta"]))
        k = r * cfg.trials
        S, R = ref["S"], ref["R"]
        if int(d[k]) == int(ref["draft"][0]):
            res["draft_equal"] += 1
        else:
            t = u[0, 0] * S
            lo = ref["cdf_w"][int(d[k]) - 1] if d[k] > 0 else 0.0
            near = min(abs(t - lo), abs(t - ref["cdf_w"][int(d[k])])) <= tol * S
            res["ambiguous_draft" if near else "mismatches"] += 1
            continue
        if bool(acc[k]) != bool(ref["accepted"][0]):
            p_d, q_d = ref["p"][int(d[k])], ref["qtilde"][int(d[k])]
            near = abs(u[0, 1] * q_d - p_d) <= tol * max(p_d, q_d)
            res["ambiguous_accept" if near else "mismatches"] += 1
            continue
        if int(o[k]) == int(ref["out_token"][0]):
            res["out_token_equal"] += 1
        else:
            t = u[0, 2] * R
            lo = ref["cdf_r"][int(o[k]) - 1] if o[k] > 0 else 0.0
            near = R > 0 and min(abs(t - lo), abs(t - ref["cdf_r"][int(o[k])])) <= tol * R
            res["ambiguous_residual" if near else "mismatches"] += 1
    res["note"] = "oracle.rdk_row on seeded rows of this run's first batch; tolerance 1e-5 of the total on CDF boundaries"
    return res


def acceptance_report(ctx: Ctx, name: str = "T1"):
    """Mean acceptance rate alpha = sum_j min(p_j, q~_j) of the three schemes of Sec. 5.2 ("Acceptance recovery") on
    the heavy-tailed extreme-pruning workload, every alpha computed by the library's kernels on the same rows:
    (a) pruning without redistribution: the unpruned drafter's q masked to the kept ids, not renormalised
        (precomputed-w mode with RDK_FLAG_W_AS_GIVEN); (b) TLI: q' at the kept ids (precomputed-w mode);
    (c) first-order RDK (the linear mode)."""
    torch, B, W = ctx.torch, ctx.B, ctx.W
    cfg = W.CONFIGS[name]
    inp = W.make_inputs(cfg, device=str(ctx.dev), with_full_drafter=True)
    kid = inp["kept_ids"].long()
    index = B.rdk_prepare_ids(inp["kept_ids"], cfg.N)
    rdk = B.rdk_sample_and_verify(index, B.RDK_MODE_LINEAR, inp["target"], inp["drafter"], None, inp["uniforms"],
                                  cfg.batch, cfg.positions)
    w = torch.zeros(cfg.rows, cfg.N, dtype=torch.float32, device=ctx.dev)
    w[:, kid] = torch.softmax(inp["drafter"].float(), dim=-1)
    tli = B.rdk_sample_and_verify(index, B.RDK_MODE_PRECOMPUTED_W, inp["target"], None, w, inp["uniforms"],
                                  cfg.batch, cfg.positions)
    q_full = torch.softmax(inp["drafter_full"].float(), dim=-1)
    w.zero_()
    w[:, kid] = q_full[:, kid]
    prune = B.rdk_sample_and_verify(index, B.RDK_MODE_PRECOMPUTED_W, inp["target"], None, w, inp["uniforms"],
                                    cfg.batch, cfg.positions, flags=B.RDK_FLAG_W_AS_GIVEN)
    torch.cuda.synchronize()
    for o in (rdk, tli, prune):
        B.check_status_word(o, f"acceptance report {name}")
    p_kept = torch.softmax(inp["target"].float(), dim=-1)[:, kid].sum(-1)
    mean = lambda t: float(t.double().mean())
    return {"workload": f"{name}: N={cfg.N}, n={cfg.n}, rows={cfg.rows}, Student-t (5 d.o.f.) logit noise, Zipf bias, bf16",
            "mean_alpha": {"pruning_without_redistribution": mean(prune["alpha"]), "tli": mean(tli["alpha"]),
                           "taylor_rdk": mean(rdk["alpha"])},
            "mean_drafter_mass_kept": mean(prune["S"]), "mean_target_mass_on_kept_ids": mean(p_kept),
            "mean_theta": mean(rdk["theta"]),
            "note": "alpha from the library's kernels (linear mode; precomputed-w mode for the two baselines); the first-order "
                    "formula moves about theta / N of the drafter's mass off the kept ids, so (b) and (c) differ by about that"}


def acceptance_exact_vs_linear(ctx: Ctx, name: str = "C5", rows: int = 256):
    """Mean acceptance rate of exact RDK (w = M^T q', Algorithm 1 step 2, bf16 affinity on the tensor cores), of the
    first-order formula (Eq. rdk-taylor) and of TLI on the same rows of the exact workload, all from the library's
    kernels; `rows` rows of the workload (the affinity matrix is the workload's own)."""
    torch, B, W = ctx.torch, ctx.B, ctx.W
    cfg = W.CONFIGS[name]
    inp = W.make_inputs(cfg, device=str(ctx.dev), with_embeddings=True)
    kind = B.RDK_PROBS if cfg.drafter_kind == "probs" else B.RDK_LOGITS
    batch = max(1, min(cfg.batch, rows // cfg.positions))
    n_rows = batch * cfg.positions
    tgt, dr, un = inp["target"][:n_rows], inp["drafter"][:n_rows], inp["uniforms"][:n_rows]
    kid = inp["kept_ids"].long()
    index = B.rdk_prepare_ids(inp["kept_ids"], cfg.N)
    M = B.rdk_build_affinity(inp["embeddings"], inp["kept_ids"], cfg.tau, B.RDK_AFF_BF16_COLS)
    w, _, _ = B.rdk_redistribute_exact(index, dr, M, batch, cfg.positions, kind)
    exact = B.rdk_sample_and_verify(index, B.RDK_MODE_PRECOMPUTED_W, tgt, None, w, un, batch, cfg.positions, kind)
    linear = B.rdk_sample_and_verify(index, B.RDK_MODE_LINEAR, tgt, dr, None, un, batch, cfg.positions, kind)
    q = dr.float() if kind == B.RDK_PROBS else torch.softmax(dr.float(), dim=-1)
    wt = torch.zeros(n_rows, cfg.N, dtype=torch.float32, device=ctx.dev)
    wt[:, kid] = q
    tli = B.rdk_sample_and_verify(index, B.RDK_MODE_PRECOMPUTED_W, tgt, None, wt, un, batch, cfg.positions, kind)
    torch.cuda.synchronize()
    for o in (exact, linear, tli):
        B.check_status_word(o, f"acceptance report {name}")
    mean = lambda t: float(t.double().mean())
    return {"workload": f"{name}: N={cfg.N}, n={cfg.n}, {n_rows} rows, affinity = soft-max of cosine similarities at tau={cfg.tau}",
            "mean_alpha": {"tli": mean(tli["alpha"]), "taylor_rdk": mean(linear["alpha"]), "exact_rdk": mean(exact["alpha"])},
            "mean_l1_exact_vs_tli": float((w / w.sum(-1, keepdim=True) - wt / wt.sum(-1, keepdim=True)).abs().sum(-1).double().mean())}


def run_ours(args):
    import torch

    import workloads as W
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (sm_100a); there is no CPU path")
    from paper_2506_03206_b200 import binding as B
    from paper_2506_03206_b200 import build
    build.build()

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    ctx = Ctx(torch, B, W, dist, dev, world, rank, local_rank, _measured_peaks())

    warmup = max(3, args.warmup)
    head = bench_workload(ctx, args.workload, args.steps, warmup, args.prior, True, not args.no_cpu_baseline)
    others = {}
    if not args.prior and not args.only:
        for name in OTHER_WORKLOADS:
            if name == args.workload:
                continue
            # the other sizes ride along with fewer steps per repeat (their steps are 4 to 10 times longer)
            k = max(3, min(args.steps, 100))
            e = bench_workload(ctx, name, k, 3, False, False, (not args.no_cpu_baseline) and W.CONFIGS[name].path == "exact")
            others[name] = {"value": e["value"], "unit": e["unit"], "ms_per_step": e["ms_per_step"], "steps": k, "timed": e["timed"],
                            "kernel_ms": e["roofline"]["kernel_ms"], "roofline": e["roofline"], "clocks": e["clocks"],
                            "config": e["config"], "gpu_launches": e["gpu_launches"]}
            if e["cpu_baseline"] is not None:
                others[name]["cpu_baseline"] = e["cpu_baseline"]
            if W.CONFIGS[name].path == "exact":
                others[name]["e2e"] = e["e2e"]
            elif e["parity"] is not None:
                others[name]["parity"] = e["parity"]
    acceptance = None
    if rank == 0 and not args.prior and (not args.only or args.workload == "T1"):
        acceptance = acceptance_report(ctx)
        if not args.only:
            acceptance["exact_vs_linear"] = acceptance_exact_vs_linear(ctx)
    if rank == 0 and args.workload == "X2":
        acceptance = {"exact_vs_linear": acceptance_exact_vs_linear(ctx, "X2", rows=W.CONFIGS["X2"].rows)}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    line = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": head["config"], "timed": head["timed"], "roofline": head["roofline"], "cpu_baseline": head["cpu_baseline"],
        "e2e": head["e2e"], "gpu_launches": head["gpu_launches"], "clocks": head["clocks"], "parity": head["parity"],
    }
    if others:
        line["workloads"] = others
    if acceptance is not None:
        line["acceptance"] = acceptance
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=["C2", "C3", "C4", "C5", "T1", "X2"], default=WORKLOAD,
                    help="the headline workload of the line (default C2, the one the metric is quoted on); the others "
                         "ride along under \"workloads\"")
    ap.add_argument("--only", action="store_true", help="time the headline workload only (profiling runs)")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the CPU checker timing (profiling runs)")
    ap.add_argument("--prior", action="store_true",
                    help="linear workloads: time the variant with a shared static prior inside Eq. rdk-taylor "
                         "(one-CTA-per-row kernel; no CPU baseline, no end-to-end leg)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
