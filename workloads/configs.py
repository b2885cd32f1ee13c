"""Seeded synthetic workloads shaped like the paper's settings.

The paper evaluates on a 128k-token vocabulary with a long-tailed token-frequency distribution
(Sec. 5.1 "Tokens"), logits whose per-position standard deviation lies between 2 and 4 (Sec. 5.1
"Logits"), drafters pruned by frequency rank (Sec. 3, Algorithm 3) down to 25 % of the vocabulary
and below ("extreme pruning", abstract).  None of its corpora or model weights are used here: every
tensor is drawn from a seeded generator with those shapes and statistics.

This module only MAKES inputs (random logits, kept-id lists, embeddings, uniforms).  It holds none
of the method's arithmetic, so the CPU checker and the CUDA library may both be fed from it.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np
import torch

from .philox import uniforms as philox_uniforms


@dataclass(frozen=True)
class RDKConfig:
    name: str
    N: int                    # target vocabulary size |T|
    n: int                    # token ids the pruned drafter keeps
    batch: int
    positions: int
    dtype: str                # "f32" | "bf16": storage type of the logits
    path: str                 # "linear" | "exact" | "both"
    kept_rule: str            # "uniform" (random n-subset) | "zipf" (n lowest frequency ranks)
    sigma: float              # logit noise scale
    zipf_bias: bool           # add b_t = -1.1 ln(rank_t) to the logits
    rho: float                # correlation of drafter and target noise on kept ids
    emb_dim: int
    trials: int
    drafter_kind: str = "logits"   # "logits" | "probs"
    tau: float = 0.1
    seed: int = 20250603
    noise: str = "normal"          # "normal" | "student_t5" (heavy-tailed logits, Sec. 5.1 "Logits")

    @property
    def rows(self) -> int:
        return self.batch * self.positions

    def with_rows(self, batch: int, positions: Optional[int] = None) -> "RDKConfig":
        return replace(self, batch=batch, positions=self.positions if positions is None else positions)


CONFIGS: Dict[str, RDKConfig] = {
    # Tiny RDK: exact and linear redistribution, 16 trials x 4 lanes = 64 uniforms per row.
    "C1": RDKConfig("C1", N=1024, n=256, batch=1, positions=4, dtype="f32", path="both",
                    kept_rule="uniform", sigma=2.0, zipf_bias=False, rho=0.0, emb_dim=64, trials=16,
                    seed=101),
    # Llama-3-scale vocabulary, 75 % pruned.
    "C2": RDKConfig("C2", N=128256, n=32064, batch=64, positions=5, dtype="bf16", path="linear",
                    kept_rule="zipf", sigma=3.0, zipf_bias=True, rho=0.0, emb_dim=256, trials=1,
                    seed=102),
    # Extreme pruning, 90 %.
    "C3": RDKConfig("C3", N=128256, n=12826, batch=256, positions=8, dtype="bf16", path="linear",
                    kept_rule="zipf", sigma=3.0, zipf_bias=True, rho=0.8, emb_dim=256, trials=1,
                    seed=103),
    # Large-vocabulary serving batch.
    "C4": RDKConfig("C4", N=262144, n=32768, batch=512, positions=4, dtype="bf16", path="linear",
                    kept_rule="zipf", sigma=3.0, zipf_bias=True, rho=0.7, emb_dim=512, trials=1,
                    seed=104),
    # Shape of the paper's synthetic acceptance experiment (Sec. 5.2): a 200k vocabulary pruned to 500
    # kept tokens, heavy-tailed (Student-t, 5 degrees of freedom) logits.  Not one of the benchmark
    # configurations; used for parity at extreme pruning and to report RDK next to TLI.
    "T1": RDKConfig("T1", N=200000, n=500, batch=32, positions=4, dtype="bf16", path="linear",
                    kept_rule="zipf", sigma=3.0, zipf_bias=True, rho=0.8, emb_dim=64, trials=1,
                    seed=106, noise="student_t5"),
    # Dense exact redistribution on tensor cores.
    "C5": RDKConfig("C5", N=32768, n=8192, batch=1024, positions=1, dtype="bf16", path="exact",
                    kept_rule="uniform", sigma=2.0, zipf_bias=False, rho=0.8, emb_dim=128, trials=1,
                    drafter_kind="probs", seed=105),
    # The exact redistribution at the Llama-3-scale shape of C2 (Sec. 4 sets it aside as O(N^2)): the
    # same vocabulary, kept ids, logits and embeddings as C2, through M^T q' instead of Eq. rdk-taylor.
    # Not one of the benchmark configurations; bench.py --workload X2 times it.
    "X2": RDKConfig("X2", N=128256, n=32064, batch=64, positions=5, dtype="bf16", path="exact",
                    kept_rule="zipf", sigma=3.0, zipf_bias=True, rho=0.0, emb_dim=256, trials=1,
                    seed=102),
}


def tiny_config(N: int = 16, n: int = 4, rows: int = 3, dtype: str = "f32", trials: int = 16,
                seed: int = 7, kept_rule: str = "uniform", rho: float = 0.5,
                drafter_kind: str = "logits", emb_dim: int = 8, zipf_bias: bool = False) -> RDKConfig:
    """A small problem for brute-force checks and edge cases (N = 2 ... a few thousand)."""
    return RDKConfig(f"tiny_N{N}_n{n}", N=N, n=n, batch=rows, positions=1, dtype=dtype, path="both",
                     kept_rule=kept_rule, sigma=2.0, zipf_bias=zipf_bias, rho=rho, emb_dim=emb_dim,
                     trials=trials, drafter_kind=drafter_kind, seed=seed)


def _torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def _gen(seed: int, device: torch.device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def token_ranks(cfg: RDKConfig) -> torch.Tensor:
    """Frequency rank (1 = most frequent) of every token id: a seeded permutation. CPU int64 [N]."""
    g = _gen(cfg.seed * 7919 + 1, torch.device("cpu"))
    perm = torch.randperm(cfg.N, generator=g)          # perm[r] = id of the token with rank r+1
    ranks = torch.empty(cfg.N, dtype=torch.int64)
    ranks[perm] = torch.arange(1, cfg.N + 1, dtype=torch.int64)
    return ranks


def kept_ids(cfg: RDKConfig) -> torch.Tensor:
    """The drafter's kept token ids, ascending, int32 [n] on the CPU."""
    if cfg.kept_rule == "zipf":
        ranks = token_ranks(cfg)
        ids = torch.nonzero(ranks <= cfg.n).flatten()
    elif cfg.kept_rule == "uniform":
        g = _gen(cfg.seed * 7919 + 2, torch.device("cpu"))
        ids = torch.randperm(cfg.N, generator=g)[: cfg.n]
    else:
        raise ValueError(cfg.kept_rule)
    return torch.sort(ids).values.to(torch.int32)


def embeddings(cfg: RDKConfig, device: str = "cpu") -> torch.Tensor:
    """Random token embeddings N(0, 1), [N, emb_dim], stored in the config's dtype."""
    dev = torch.device(device)
    g = _gen(cfg.seed * 7919 + 3, dev)
    e = torch.randn(cfg.N, cfg.emb_dim, generator=g, device=dev, dtype=torch.float32)
    return e.to(_torch_dtype(cfg.dtype))


def make_inputs(cfg: RDKConfig, device: str = "cpu", variant: int = 0,
                with_embeddings: bool = False, row_chunk: int = 128,
                with_full_drafter: bool = False) -> Dict[str, object]:
    """Draw one batch of inputs for ``cfg``.

    Returns a dict with
      kept_ids  int32 [n] (device)            ascending target-token ids the drafter keeps
      target    dtype [rows, N]               target logits z
      drafter   dtype [rows, n]               drafter logits y (or probabilities, C5)
      uniforms  float32 [rows, trials, 4]     Philox uniforms
      embeddings dtype [N, emb_dim]           only when with_embeddings
      drafter_full dtype [rows, N]            only when with_full_drafter (logit workloads): the logits of
                                              the drafter before pruning, equal to ``drafter`` at the kept ids
    ``variant`` selects an independent batch of the same workload (used to rotate buffers).
    """
    dev = torch.device(device)
    dt = _torch_dtype(cfg.dtype)
    rows, N, n = cfg.rows, cfg.N, cfg.n
    kid_cpu = kept_ids(cfg)
    kid = kid_cpu.to(dev)
    kidl = kid.long()
    if cfg.zipf_bias:
        bias = (-1.1 * torch.log(token_ranks(cfg).to(torch.float32))).to(dev)
    else:
        bias = torch.zeros(N, dtype=torch.float32, device=dev)
    g = _gen(cfg.seed * 7919 + 11 + 1000003 * variant, dev)
    target = torch.empty(rows, N, dtype=dt, device=dev)
    drafter = torch.empty(rows, n, dtype=dt, device=dev)
    c = math.sqrt(max(0.0, 1.0 - cfg.rho * cfg.rho))
    if with_full_drafter and cfg.drafter_kind == "probs":
        raise ValueError("with_full_drafter is defined for the logit workloads only")
    # the pruned-away part of the drafter comes from a generator of its own, so that asking for it
    # leaves every other tensor of the batch as it was
    g_full = _gen(cfg.seed * 7919 + 13 + 1000003 * variant, dev) if with_full_drafter else None
    drafter_full = torch.empty(rows, N, dtype=dt, device=dev) if with_full_drafter else None
    def noise(*shape, gen=None):
        gen = g if gen is None else gen
        x = torch.randn(*shape, generator=gen, device=dev, dtype=torch.float32)
        if cfg.noise == "student_t5":     # t_5 = normal / sqrt(chi2_5 / 5), rescaled to unit variance (var of t_5 is 5/3)
            chi2 = torch.zeros(*shape, device=dev, dtype=torch.float32)
            for _ in range(5):
                chi2 += torch.randn(*shape, generator=gen, device=dev, dtype=torch.float32) ** 2
            x = x / torch.sqrt(chi2 / 5.0) * math.sqrt(3.0 / 5.0)
        return x

    for r0 in range(0, rows, row_chunk):
        r1 = min(rows, r0 + row_chunk)
        gz = noise(r1 - r0, N)
        h = noise(r1 - r0, n)
        if cfg.drafter_kind == "probs":
            # C5 recipe: the drafter is drawn first, the target copies a correlated part of it.
            y = cfg.sigma * h
            h2 = torch.randn(r1 - r0, n, generator=g, device=dev, dtype=torch.float32)
            z = cfg.sigma * gz + bias
            z[:, kidl] = cfg.rho * y + cfg.sigma * c * h2 + bias[kidl]
            target[r0:r1] = z.to(dt)
            drafter[r0:r1] = torch.softmax(y, dim=-1).to(dt)
        else:
            z = bias + cfg.sigma * gz
            y = bias[kidl] + cfg.sigma * (cfg.rho * gz[:, kidl] + c * h)
            target[r0:r1] = z.to(dt)
            drafter[r0:r1] = y.to(dt)
            if with_full_drafter:
                yf = bias + cfg.sigma * (cfg.rho * gz + c * noise(r1 - r0, N, gen=g_full))
                yf[:, kidl] = y
                drafter_full[r0:r1] = yf.to(dt)
    u = torch.from_numpy(philox_uniforms(cfg.seed + 104729 * variant, rows, cfg.trials)).to(dev)
    out: Dict[str, object] = {"cfg": cfg, "kept_ids": kid, "target": target, "drafter": drafter,
                              "uniforms": u}
    if with_embeddings:
        out["embeddings"] = embeddings(cfg, device)
    if with_full_drafter:
        out["drafter_full"] = drafter_full
    return out


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Widen a tensor exactly (f32 / bf16 -> f64) into a numpy array on the host."""
    return t.detach().to("cpu").to(torch.float64).numpy()
