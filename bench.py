"""Benchmark of the RDK hot path on B200.

One "step" takes one batch of the Llama-3-scale workload (target vocabulary N = 128256, drafter
keeps n = 32064 ids, 64 sequences x 5 draft positions = 320 rows, bf16 logits) through the whole
path: drafter/target soft-max, Token-Level Intersection, first-order redistribution, draft draw,
rejection test, acceptance rate, residual draw and the per-sequence accepted length.  The metric
is verified draft tokens per second = rows x steps / elapsed.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  With --impl reference the CPU checker (oracle/) is timed on the host cores
instead; that arm touches no GPU.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOAD = "C2"              # default: the configuration the metric is quoted on (--workload picks another)
N_BUFFER_SETS = 6            # distinct input batches rotated through, so every step reads HBM
METRIC = "verified draft tokens/sec"
UNIT = "tokens/s"

# DRAM traffic of one launch of the dominant kernel from an ncu capture
# (dram__bytes_read.sum + dram__bytes_write.sum), valid only for the kernel sources with this hash.
NCU_TRAFFIC = {"sources_sha256": "368495009f2b0618217eb5ae984b3a808be9932e751962e2c1759995890eed39",
               "bytes_per_launch": 102941952 + 3496704}   # rdk_stream_kernel, profiles/rdk_stream_and_draw_kernels_C2.md
KERNEL_SOURCES = ("rdk_row_stream.cu", "rdk_row.cuh", "rdk_common.cuh")


def _kernel_sources_hash() -> str:
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2506_03206_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


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

    def summary(self):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["nvml unavailable"]}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


def _cpu_baseline(cfg, min_seconds: float = 10.0, pool_rows: int = 64):
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
    return done / dt, dt, done


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


def _peak_tensor():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["bf16_tflops"]), float(d["bf16_tflops_sustained"]), "measured (MEASURED_PEAKS.json bf16_tflops, burst)"
    return 1590.0, 1400.0, "fallback (1.59 PFLOP/s burst, earlier measurement on this pool)"


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

    cfg = W.CONFIGS[args.workload]
    exact = cfg.path == "exact"
    rows, trials = cfg.rows, cfg.trials
    zb = 2 if cfg.dtype == "bf16" else 4
    kind = B.RDK_PROBS if cfg.drafter_kind == "probs" else B.RDK_LOGITS
    row_bytes = cfg.N * zb + cfg.n * zb + trials * 16 + 30
    # enough distinct batches that one rotation exceeds L2 several times over (C5's operands do so alone)
    nsets = 1 if exact else max(2, min(N_BUFFER_SETS, int(600e6 // (rows * row_bytes)) + 1))
    sets = [W.make_inputs(cfg, device=str(dev), variant=v + 100 * rank, with_embeddings=exact and v == 0)
            for v in range(nsets)]
    index = B.rdk_prepare_ids(sets[0]["kept_ids"], cfg.N)
    outs = [B.alloc_outputs(rows, cfg.batch, trials, dev) for _ in range(nsets)]
    outs_nolen = [{k: v for k, v in o.items() if k != "accepted_len"} for o in outs]
    pb = B.make_problem(index, sets[0]["target"], sets[0]["drafter"], cfg.batch, cfg.positions, kind)
    ws = B.sample_workspace(pb, B.RDK_MODE_LINEAR, trials, dev)

    prep_ms = None
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
        launches_per_step = 2 + 2          # operand, contraction; row kernel, accepted length
    elif args.prior:
        # Eq. rdk-taylor with one shared prior row (a static stand-in for the unknown target distribution)
        shared_prior = sets[-1]["target"][0].clone().contiguous()

        def step(i, out_list=outs):
            s = sets[i % nsets]
            B.rdk_sample_and_verify_prior(index, s["target"], shared_prior, s["drafter"], s["uniforms"],
                                          cfg.batch, cfg.positions, kind, out=out_list[i % nsets])
        launches_per_step = 2              # row kernel, accepted length
    else:
        def step(i, out_list=outs):
            s = sets[i % nsets]
            B.rdk_sample_and_verify(index, B.RDK_MODE_LINEAR, s["target"], s["drafter"], None, s["uniforms"],
                                    cfg.batch, cfg.positions, kind, out=out_list[i % nsets], ws=ws)
        launches_per_step = 2              # stream kernel, draw kernel

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(fn, n_steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for i in range(n_steps):
            fn(i)
        e1.record()
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), dist, dev)

    warmup = max(3, args.warmup)
    for i in range(warmup):
        step(i)
    sampler = ClockSampler(local_rank)
    sampler.start()
    ms = timed(step, args.steps)
    # the dominant kernels alone: linear = stream + draw kernels (no accepted length); exact = the
    # contraction call (operand preparation, tensor-core kernel, row sums)
    ms_kernel = timed(contraction if exact else (lambda i: step(i, outs_nolen)), args.steps)
    sampler.stop()
    sampler.join(timeout=1.0)
    B.check_status_word(outs[0], "bench step")

    e2e = None
    if not exact and not args.prior:
        # end to end: host (pinned) buffers in, host results out, copies inside the timed region
        e2e_steps = max(3, min(args.steps, 20))
        host_sets = [{k: s[k].cpu().pin_memory() for k in ("target", "drafter", "uniforms")} for s in sets[:2]]
        stage = {"target": torch.empty_like(sets[0]["target"]), "drafter": torch.empty_like(sets[0]["drafter"]),
                 "uniforms": torch.empty_like(sets[0]["uniforms"]), "ws": ws}
        host_out = {k: torch.empty_like(v, device="cpu").pin_memory() for k, v in outs[0].items() if not k.startswith("_")}

        def e2e_step(i):
            h = host_sets[i % len(host_sets)]
            B.rdk_sample_and_verify_host(index, h["target"], h["drafter"], h["uniforms"], cfg.batch, cfg.positions,
                                         stage, outs[0], host_out, kind)

        for i in range(3):
            e2e_step(i)
        ms_e2e = timed(e2e_step, e2e_steps)
        h2d = sum(host_sets[0][k].numel() * host_sets[0][k].element_size() for k in ("target", "drafter", "uniforms"))
        d2h = sum(v.numel() * v.element_size() for v in host_out.values())
        e2e = {"value": world * rows * trials * e2e_steps / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    value = whole_job_value(rows, trials, args.steps, world, ms)
    kernel_ms = ms_kernel / args.steps
    if exact:
        peak, peak_sus, peak_src = _peak_tensor()
        flops = 2.0 * rows * cfg.n * cfg.N
        achieved = flops / (kernel_ms * 1e-3) / 1e12
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                    "traffic": None, "kernel_ms": kernel_ms, "flops_per_launch": flops, "peak_source": peak_src,
                    "frac_of_sustained_peak": achieved / peak_sus,
                    "kernels": "exact_operand_kernel + exact_tc_kernel (row sums in its epilogue)"}
    else:
        peak, peak_src = _peaks()
        algo_bytes = rows * row_bytes
        achieved = algo_bytes / (kernel_ms * 1e-3) / 1e9
        traffic = NCU_TRAFFIC["bytes_per_launch"] if (args.workload == WORKLOAD and
                                                      NCU_TRAFFIC["sources_sha256"] == _kernel_sources_hash()) else None
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "traffic": traffic, "kernel_ms": kernel_ms, "algorithmic_bytes_per_launch": algo_bytes,
                    "peak_source": peak_src,
                    "kernels": "rdk_row_kernel (shared prior)" if args.prior else "rdk_stream_kernel + rdk_draw_kernel"}
        if args.prior:
            roofline["traffic"] = None

    cpu = None
    if not args.no_cpu_baseline and not exact and not args.prior:
        cpu_value, cpu_dt, cpu_rows = _cpu_baseline(cfg)
        cpu = {"value": cpu_value, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"{cpu_rows} rows of {args.workload} through oracle.rdk_row (float64 numpy, one thread, {cpu_dt:.1f} s)"}

    what = ("exact RDK on tensor cores (bf16 affinity, fp32 accumulate) + sampling/verification" if exact
            else "linear RDK with one shared prior row in Eq. rdk-taylor + sampling/verification" if args.prior
            else "linear RDK (first-order redistribution + sampling/verification)")
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {what}, N={cfg.N}, n={cfg.n}, batch={cfg.batch}, "
                               f"positions={cfg.positions} (rows={rows}), bf16 inputs, trials={trials}",
                   "rows_per_step": rows, "parallelism": f"replicas x{world} (no collective)",
                   "l2": (f"operands of one step ({(cfg.N * cfg.n * 2 + rows * cfg.N * 4) / 1e6:.0f} MB) exceed the 126 MB L2"
                          if exact else
                          f"inputs rotate over {nsets} distinct batches ({nsets * rows * row_bytes / 1e6:.0f} MB > 126 MB L2)")},
        "roofline": roofline,
        "cpu_baseline": cpu,
        "e2e": e2e,
        "gpu_launches": launches_per_step * args.steps,
        "clocks": sampler.summary(),
    }
    if prep_ms is not None:
        line["config"]["preprocessing_ms"] = prep_ms
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=["C2", "C3", "C4", "C5"], default=WORKLOAD,
                    help="C2 (default) is the benchmark; C3/C4 are the other linear-path sizes, C5 the exact "
                         "tensor-core path (used for profiling)")
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
