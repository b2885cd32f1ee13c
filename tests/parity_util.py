"""Helpers that compare the CUDA library's outputs with the CPU checker, row by row."""
from __future__ import annotations

import json
import math
import os
from typing import Dict, Iterable, Optional

import numpy as np
import torch

from oracle import rdk_oracle as O
from workloads import to_f64

# Tolerances: max abs error 1e-5 on probabilities / acceptance probabilities for fp32 inputs and
# 2e-3 relative for bf16 inputs.  bf16 inputs are exact values for both sides and the kernels
# compute in fp32 either way, so the fp32 absolute bound is applied to both; the relative bound is
# applied on top for bf16.
ABS_TOL = 1e-5
REL_TOL_BF16 = 2e-3
BOUNDARY_TOL = 1e-5      # a draw is "ambiguous" when u * total is this close (relative to total) to
                         # the CDF interval of the token the GPU picked


def close(gpu: float, ref: float, bf16: bool) -> bool:
    if abs(gpu - ref) > ABS_TOL:
        return False
    if bf16 and abs(gpu - ref) > REL_TOL_BF16 * abs(ref) + 1e-30:
        return False
    return True


def interval_distance(cdf: np.ndarray, tok: int, t: float) -> float:
    """Distance of the threshold t from token tok's CDF interval [C_{tok-1}, C_tok]."""
    lo = cdf[tok - 1] if tok > 0 else 0.0
    hi = cdf[tok]
    if t < lo:
        return lo - t
    if t > hi:
        return t - hi
    return 0.0


class Tally:
    def __init__(self):
        self.rows = 0
        self.draws = 0
        self.ambiguous_draft = 0
        self.ambiguous_accept = 0
        self.ambiguous_residual = 0
        self.failures = []
        self.max_abs = {}

    def err(self, name: str, gpu: float, ref: float):
        self.max_abs[name] = max(self.max_abs.get(name, 0.0), abs(gpu - ref))

    def fail(self, msg: str):
        self.failures.append(msg)

    def summary(self) -> str:
        return (f"rows={self.rows} draws={self.draws} ambiguous(draft/accept/residual)="
                f"{self.ambiguous_draft}/{self.ambiguous_accept}/{self.ambiguous_residual} "
                f"max_abs={ {k: float('%.3g' % v) for k, v in self.max_abs.items()} } "
                f"failures={len(self.failures)}")

    def assert_ok(self, max_ambiguous_frac: float = 0.05):
        assert not self.failures, self.summary() + "\n" + "\n".join(self.failures[:20])
        amb = self.ambiguous_draft + self.ambiguous_accept + self.ambiguous_residual
        assert amb <= max(2, max_ambiguous_frac * self.draws), self.summary()

    def assert_ok_at_scale(self, n: int):
        """Full-size runs: the library's prefix sums are fp32 inside a segment and fp64 across segments
        (absolute error about 1e-7 of the total), so a draw's threshold falls that close to one of the
        about 2 n interval ends that matter with probability 2 n 1e-7; three times that expectation,
        rounded up, is allowed, never a fixed fraction of the draws."""
        assert not self.failures, self.summary() + "\n" + "\n".join(self.failures[:20])
        amb = self.ambiguous_draft + self.ambiguous_accept + self.ambiguous_residual
        allowed = math.ceil(3.0 * 2.0 * n * 1e-7 * self.draws)
        assert amb <= allowed, f"{amb} ambiguous draws, {allowed} allowed: " + self.summary()

    def record(self, name: str):
        """Keep the tally: one JSON line per comparison in parity_tallies.jsonl (next to the other run
        outputs when that folder exists, else in the working directory), and on stdout."""
        line = {"case": name, "rows": self.rows, "draws": self.draws, "ambiguous_draft": self.ambiguous_draft,
                "ambiguous_accept": self.ambiguous_accept, "ambiguous_residual": self.ambiguous_residual,
                "failures": len(self.failures), "max_abs": {k: float("%.3g" % v) for k, v in self.max_abs.items()}}
        root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
        folder = os.path.join(root, "gpurun_out")
        path = os.path.join(folder if os.path.isdir(folder) else os.getcwd(), "parity_tallies.jsonl")
        try:
            with open(path, "a") as f:
                f.write(json.dumps(line) + "\n")
        except OSError:
            pass
        print("parity tally:", json.dumps(line))


def compare_sampling(inp: Dict[str, object], out: Dict[str, torch.Tensor], rows: Iterable[int],
                     mode: str, tally: Optional[Tally] = None, M: Optional[np.ndarray] = None,
                     w_given: Optional[np.ndarray] = None, operand_bf16: bool = False,
                     kept_ids: Optional[np.ndarray] = None, prior=None) -> Tally:
    """Compare rdk_sample_and_verify outputs against the checker for the given rows.

    inp: the generator's dict (target, drafter, uniforms, cfg, kept_ids); tensors may live on the GPU.
    mode: "linear" | "exact" | "given" as in the checker's rdk_row.
    w_given: [len(rows), N] float64 when mode == "given".
    """
    cfg = inp["cfg"]
    bf16 = cfg.dtype == "bf16"
    tally = tally or Tally()
    kappa = (kept_ids if kept_ids is not None else inp["kept_ids"].cpu().numpy()).astype(np.int64)
    o = {k: v.detach().cpu().numpy() for k, v in out.items() if v is not None}
    trials = inp["uniforms"].shape[1]
    for idx, r in enumerate(rows):
        z = to_f64(inp["target"][r])
        y = to_f64(inp["drafter"][r]) if inp.get("drafter") is not None else None
        u = inp["uniforms"][r].cpu().numpy().astype(np.float64)
        pr = None if prior is None else to_f64(prior if prior.dim() == 1 else prior[r])
        ref = O.rdk_row(z, y, kappa, u, mode, M=M, drafter_kind=cfg.drafter_kind, operand_bf16=operand_bf16,
                        w_given=None if w_given is None else w_given[idx], prior=pr)
        tally.rows += 1
        for name, key in (("alpha", "alpha"), ("S", "S"), ("residual_mass", "R")):
            g = float(o[name][r])
            tally.err(name, g, ref[key])
            # S is a total weight (about 1); alpha and R are probabilities
            if not close(g, ref[key], bf16):
                tally.fail(f"row {r}: {name} gpu={g!r} ref={ref[key]!r}")
        if mode == "linear":
            g = float(o["theta"][r])
            tally.err("theta", g, ref["theta"])
            if not close(g, ref["theta"], bf16):
                tally.fail(f"row {r}: theta gpu={g!r} ref={ref['theta']!r}")
        S, R = ref["S"], ref["R"]
        p, qt = ref["p"], ref["qtilde"]
        for t in range(trials):
            k = r * trials + t
            tally.draws += 1
            d_g, d_r = int(o["draft_token"][k]), int(ref["draft"][t])
            if not (0 <= d_g < cfg.N):
                tally.fail(f"row {r} trial {t}: draft token {d_g} out of range")
                continue
            if d_g != d_r:
                dist = interval_distance(ref["cdf_w"], d_g, u[t, 0] * S)
                if dist <= BOUNDARY_TOL * S and ref["w"][d_g] > 0:
                    tally.ambiguous_draft += 1
                else:
                    tally.fail(f"row {r} trial {t}: draft gpu={d_g} ref={d_r} dist={dist:.3e}")
                continue                       # a different (valid) draft: the rest is not comparable
            a_g = float(o["accept_prob"][k])
            tally.err("accept_prob", a_g, ref["accept_prob"][t])
            if not close(a_g, ref["accept_prob"][t], bf16):
                tally.fail(f"row {r} trial {t}: accept_prob gpu={a_g!r} ref={ref['accept_prob'][t]!r}")
            acc_g, acc_r = bool(o["accepted"][k]), bool(ref["accepted"][t])
            if acc_g != acc_r:
                margin = abs(u[t, 1] * qt[d_r] - p[d_r])
                if margin <= BOUNDARY_TOL * max(p[d_r], qt[d_r]):
                    tally.ambiguous_accept += 1
                else:
                    tally.fail(f"row {r} trial {t}: accepted gpu={acc_g} ref={acc_r} margin={margin:.3e}")
                continue
            out_g = int(o["out_token"][k])
            if acc_r:
                if out_g != d_r:
                    tally.fail(f"row {r} trial {t}: accepted but out_token {out_g} != draft {d_r}")
                continue
            t_r = int(ref["residual_token"][t])
            if out_g != t_r:
                if R > 0:
                    dist = interval_distance(ref["cdf_r"], out_g, u[t, 2] * R) if 0 <= out_g < cfg.N else np.inf
                    ok = dist <= BOUNDARY_TOL * R and ref["r"][out_g] > 0
                else:
                    ok = False
                if ok:
                    tally.ambiguous_residual += 1
                else:
                    tally.fail(f"row {r} trial {t}: residual token gpu={out_g} ref={t_r}")
    return tally


def compare_accepted_len(out: Dict[str, torch.Tensor], batch: int, positions: int, trials: int) -> None:
    """accepted_len must equal the checker's count applied to the GPU's own accept flags."""
    acc = out["accepted"].cpu().numpy().reshape(batch, positions, trials).astype(bool)
    got = out["accepted_len"].cpu().numpy().reshape(batch, trials)
    for t in range(trials):
        want = O.accepted_len(acc[:, :, t])
        assert np.array_equal(got[:, t], want)


def compare_qtilde(qt_gpu: torch.Tensor, ref_rows: Dict[int, dict], bf16: bool) -> float:
    worst = 0.0
    for r, ref in ref_rows.items():
        g = qt_gpu[r].cpu().numpy().astype(np.float64)
        diff = np.abs(g - ref["qtilde"])
        worst = max(worst, float(diff.max()))
        assert diff.max() <= ABS_TOL, f"row {r}: q~ max abs error {diff.max():.3e}"
        if bf16:
            rel = diff / np.maximum(ref["qtilde"], 1e-30)
            sel = ref["qtilde"] > 1e-30
            assert rel[sel].max() <= REL_TOL_BF16, f"row {r}: q~ max rel error {rel[sel].max():.3e}"
        assert abs(g.sum() - 1.0) < 1e-4 and (g >= 0).all()
    return worst
