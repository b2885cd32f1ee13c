"""CPU checker for the Redistributing-Drafter-Kernels (RDK) sampler -- TEST INFRASTRUCTURE ONLY.

This file is a plain, slow, float64 numpy transcription of what the paper defines, one row
(sequence, draft position) at a time, in the paper's order and notation.  It exists so that the
CUDA library can be compared against something that a reader can check against the paper by eye.
It is NOT part of the product: only the tests, the smoke check and the benchmark's CPU-baseline
leg may import it, and it shares no code with the CUDA path (it imports numpy and nothing else).

Notation (the paper reuses symbols; one name per object here):
  N      target vocabulary size |T|                       (Theorem 4.4: N = |T|)
  n      number of token ids the pruned drafter keeps
  kappa  kept ids, drafter index i -> target token id     (the intersection I = T n D, Sec. 2)
  p      target distribution, length N
  q      drafter distribution over its n kept tokens
  q'     q after Token-Level Intersection (Eq. tli-drafter): length N, zero off I, sums to 1
  M      row-stochastic token-affinity matrix, n x N      (Eq. symbolic-m, rows i in I)
  w      un-normalised redistributed weights (the paper's p-tilde), S = sum_j w_j
  q~     redistributed drafter distribution w / S          (the paper's p', p_RDK, p_Taylor)
  theta  p^T q'                                            (Sec. 4, defined just before Eq. rdk-taylor)
  alpha  acceptance rate sum_x min(p(x), q~(x))            (Definition 2.1)

Conventions the paper leaves open and this checker fixes (each is a documented reading):
  * "Sample" (Algorithm 4) is inverse-CDF in ascending token id: the smallest j whose inclusive
    prefix sum C_j is strictly greater than u * C_last, u in [0, 1).  A zero-weight token can
    never be drawn.  If rounding leaves no such j, the last positive-weight token is taken.
  * The rejection test of Algorithm 4 (a draft with p below q~ is turned down with the
    complementary probability of p / q~) is taken as:  accepted  <=>  u2 * q~(d) < p(d).
  * The residual normaliser 1 - sum min(p, q~) is computed as the direct sum of max(0, p - q~);
    if that sum is not positive the replacement token is drawn from p.
  * kept ids < 0 or >= N stand for drafter tokens outside the target vocabulary (the set F of
    Sec. 2); the TLI step drops them.

Pins (tests/test_oracle_pins.py, `-m "not gpu"`), per function:
  softmax            Theorem 4.2 bound, shift invariance, equal logits -> uniform
  round_to_bf16      exhaustive agreement with the IEEE bit pattern rule on a grid of values
  tli_project        Eq. tli-drafter by hand on a 5-token case; invalid ids re-spread
  build_affinity     rows >= 0 and sum to 1 (Assumption 4.1); tau -> inf gives 1/N; tau -> 0
                     gives the identity on the kept rows; orthonormal embeddings closed form;
                     Lemma (non-expansive) inequality
  redistribute_exact identity M -> q' (RDK = TLI); m = 2 worked example of Theorem 4.3;
                     Theorem 4.1 inequality; double loop at N <= 16
  redistribute_linear uniform p closed form (theta = 1/N, S = 1, OOV mass 1/(N^3+N) each);
                     Theorem 4.4 regime test; hand rationals at N = 4
  inverse_cdf        sweep of u over interval midpoints and both sides of every boundary
  accept_test / residual / acceptance_rate
                     exact enumeration at N <= 16: sum_d q~_d a_d = alpha and
                     q~_t a_t + (1 - alpha) r_t = p_t for every t (output distributed as p);
                     Lemma 2.3 alpha = 1 - ||k||_1 = 1 - 0.5 ||p - q~||_1; Monte-Carlo
  accepted_len       brute force over all accept patterns
  emit_sequence      brute force over all accept patterns; bonus draw frequency against p
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


class EmptyIntersection(ValueError):
    """No kept id lies in the target vocabulary (the paper assumes I is non-empty, Sec. 2)."""


class BadIds(ValueError):
    """Two drafter indices map to the same target token."""


# ----------------------------------------------------------------------------------------------
# O1  softmax (Sec. 4.1, the display below Eq. "logits")
# ----------------------------------------------------------------------------------------------
def softmax(z: np.ndarray) -> np.ndarray:
    """p_i = exp(z_i) / sum_j exp(z_j); the row maximum is subtracted first (same value)."""
    z = np.asarray(z, dtype=F64)
    e = np.exp(z - np.max(z))
    return e / np.sum(e)


# ----------------------------------------------------------------------------------------------
# storage rounding used when an operand is kept in bfloat16 (not from the paper; the paper never
# states a precision).  Round-to-nearest-even on an 8-bit significand, done on the float64 value.
# ----------------------------------------------------------------------------------------------
def round_to_bf16(x: np.ndarray) -> np.ndarray:
    x = np.asarray(x, dtype=F64)
    _, e = np.frexp(x)                       # x = m * 2**e with 0.5 <= |m| < 1
    q = np.maximum(e - 8, -133)              # exponent of one unit in the last place
    scale = np.ldexp(1.0, q)
    return np.rint(x / scale) * scale        # np.rint rounds halves to even


# ----------------------------------------------------------------------------------------------
# O2  Token-Level Intersection (Eq. tli-drafter; Algorithm 1 step 1; Algorithm 2 step 1)
# ----------------------------------------------------------------------------------------------
def tli_project(q: np.ndarray, kappa: np.ndarray, N: int) -> np.ndarray:
    """Scatter q to length N, drop entries whose id is outside the target vocabulary, and
    renormalise over the intersection.  Returns q' (length N)."""
    q = np.asarray(q, dtype=F64)
    kappa = np.asarray(kappa, dtype=np.int64)
    valid = (kappa >= 0) & (kappa < N)
    if not np.any(valid):
        raise EmptyIntersection("no kept id inside the target vocabulary")
    ids = kappa[valid]
    if np.unique(ids).size != ids.size:
        raise BadIds("duplicate kept id")
    qhat = np.zeros(N, dtype=F64)
    qhat[ids] = q[valid]
    return qhat / np.sum(qhat)


# ----------------------------------------------------------------------------------------------
# O0  token-affinity matrix (Eq. symbolic-m), with Omega = cosine similarity of embeddings
# ----------------------------------------------------------------------------------------------
def build_affinity(E: np.ndarray, kappa: np.ndarray, tau: float,
                   row_block: int = 512) -> np.ndarray:
    """M_ij = exp(Omega_ij / tau) / sum_{k in T} exp(Omega_ik / tau), i in I, j in T, with
    Omega_ij = <e_kappa_i, e_j> / (|e_kappa_i| |e_j|).  The sum runs over ALL k in T, k = kappa_i
    included.  Rows whose id is outside the vocabulary are left zero (never used).  [n, N]."""
    E = np.asarray(E, dtype=F64)
    kappa = np.asarray(kappa, dtype=np.int64)
    N = E.shape[0]
    norms = np.maximum(np.sqrt(np.sum(E * E, axis=1)), 1e-12)
    Eh = E / norms[:, None]
    M = np.zeros((kappa.size, N), dtype=F64)
    for i0 in range(0, kappa.size, row_block):
        ids = kappa[i0:i0 + row_block]
        ok = (ids >= 0) & (ids < N)
        omega = Eh[np.where(ok, ids, 0)] @ Eh.T                 # [block, N]
        a = omega / tau
        a = np.exp(a - np.max(a, axis=1, keepdims=True))
        a = a / np.sum(a, axis=1, keepdims=True)
        a[~ok] = 0.0
        M[i0:i0 + row_block] = a
    return M


def affinity_columns(E: np.ndarray, kappa: np.ndarray, tau: float, cols: np.ndarray,
                     row_block: int = 1024) -> np.ndarray:
    """The same matrix as build_affinity, but only the requested columns are kept ([n, len(cols)]).
    The row normaliser still runs over all of T.  For sizes whose full matrix is too big to hold."""
    E = np.asarray(E, dtype=F64)
    kappa = np.asarray(kappa, dtype=np.int64)
    cols = np.asarray(cols, dtype=np.int64)
    N = E.shape[0]
    norms = np.maximum(np.sqrt(np.sum(E * E, axis=1)), 1e-12)
    Eh = E / norms[:, None]
    out = np.zeros((kappa.size, cols.size), dtype=F64)
    for i0 in range(0, kappa.size, row_block):
        ids = kappa[i0:i0 + row_block]
        ok = (ids >= 0) & (ids < N)
        a = (Eh[np.where(ok, ids, 0)] @ Eh.T) / tau
        a = np.exp(a - np.max(a, axis=1, keepdims=True))
        blk = a[:, cols] / np.sum(a, axis=1, keepdims=True)
        blk[~ok] = 0.0
        out[i0:i0 + row_block] = blk
    return out


# ----------------------------------------------------------------------------------------------
# O3e  exact redistribution (Algorithm 1 step 2:  p' = M^T q')
# ----------------------------------------------------------------------------------------------
def redistribute_exact(qprime_kept: np.ndarray, M: np.ndarray) -> np.ndarray:
    """w_j = sum_i q'_{kappa_i} M_ij.  qprime_kept holds q' at the kept ids (length n)."""
    return np.asarray(qprime_kept, dtype=F64) @ np.asarray(M, dtype=F64)


def redistribute_exact_loops(qprime_kept, M) -> np.ndarray:
    """The definition as a literal double loop (small sizes only)."""
    n, N = M.shape
    w = np.zeros(N, dtype=F64)
    for j in range(N):
        acc = 0.0
        for i in range(n):
            acc += float(qprime_kept[i]) * float(M[i, j])
        w[j] = acc
    return w


# ----------------------------------------------------------------------------------------------
# O3l  first-order redistribution (Eq. rdk-taylor)
# ----------------------------------------------------------------------------------------------
def redistribute_linear(p: np.ndarray, qprime: np.ndarray):
    """theta = p^T q';  w_j = (N q'_j + theta p_j) / (N + p_j), N = |T| as a real number.
    Returns (theta, w)."""
    p = np.asarray(p, dtype=F64)
    qprime = np.asarray(qprime, dtype=F64)
    N = float(p.size)
    theta = float(np.dot(p, qprime))
    w = (N * qprime + theta * p) / (N + p)
    return theta, w


# ----------------------------------------------------------------------------------------------
# O4  normalisation  (Eq. rdk-taylor, second part;  Algorithm 1 step 2: the weights are scaled to sum to 1)
# ----------------------------------------------------------------------------------------------
def normalise(w: np.ndarray):
    """S = sum_j w_j (ascending j), q~ = w / S.  Returns (S, q~)."""
    w = np.asarray(w, dtype=F64)
    S = float(np.cumsum(w)[-1])
    return S, w / S


# ----------------------------------------------------------------------------------------------
# O5  categorical draw (Algorithm 4 step 2 "Sample"; the convention is this checker's reading)
# ----------------------------------------------------------------------------------------------
def inverse_cdf(weights: np.ndarray, u: float) -> int:
    weights = np.asarray(weights, dtype=F64)
    C = np.cumsum(weights)
    t = float(u) * C[-1]
    j = int(np.searchsorted(C, t, side="right"))        # first j with C_j > t
    if j >= weights.size:
        pos = np.nonzero(weights > 0)[0]
        j = int(pos[-1]) if pos.size else weights.size - 1
    return j


# ----------------------------------------------------------------------------------------------
# O6  rejection test (Algorithm 4 steps 5-7)
# ----------------------------------------------------------------------------------------------
def accept_test(p: np.ndarray, qt: np.ndarray, d: int, u2: float):
    """a = min(1, p_d / q~_d); accepted <=> u2 * q~_d < p_d.  Returns (a, accepted)."""
    pd, qd = float(p[d]), float(qt[d])
    a = 1.0 if pd >= qd else pd / qd
    return a, bool(float(u2) * qd < pd)


# ----------------------------------------------------------------------------------------------
# O7  acceptance rate (Definition 2.1)
# ----------------------------------------------------------------------------------------------
def acceptance_rate(p: np.ndarray, qt: np.ndarray) -> float:
    return float(np.sum(np.minimum(p, qt)))


# ----------------------------------------------------------------------------------------------
# O8  residual distribution (Algorithm 4 step 8; Definition 2.2 with the roles of p, q swapped)
# ----------------------------------------------------------------------------------------------
def residual(p: np.ndarray, qt: np.ndarray):
    """r_j = max(0, p_j - q~_j), R = sum_j r_j.  Returns (R, r) with r un-normalised."""
    r = np.maximum(0.0, np.asarray(p, dtype=F64) - np.asarray(qt, dtype=F64))
    return float(np.cumsum(r)[-1]), r


def residual_sample(p: np.ndarray, qt: np.ndarray, u3: float) -> int:
    R, r = residual(p, qt)
    if R > 0.0:
        return inverse_cdf(r, u3)
    return inverse_cdf(p, u3)


# ----------------------------------------------------------------------------------------------
# O9  number of accepted drafts per sequence (Algorithm 4 step 7)
# ----------------------------------------------------------------------------------------------
def accepted_len(accepted: np.ndarray) -> np.ndarray:
    """accepted: bool [batch, positions] -> int32 [batch], the count of leading True values."""
    accepted = np.asarray(accepted, dtype=bool)
    out = np.zeros(accepted.shape[0], dtype=np.int32)
    for b in range(accepted.shape[0]):
        k = 0
        while k < accepted.shape[1] and accepted[b, k]:
            k += 1
        out[b] = k
    return out


# ----------------------------------------------------------------------------------------------
# O10  the emitted sequence (Algorithm 4 steps 7-9): the accepted drafts d_1..d_j followed by one
#      more token t: the residual draw made where the first rejection happened, or, if every draft
#      was accepted, a fresh draw t ~ p from the target row that follows the last draft
# ----------------------------------------------------------------------------------------------
def emit_sequence(draft, accepted, out_token, p_bonus, u_bonus) -> list:
    """draft, accepted, out_token: per draft position of ONE sequence (out_token[k] is the residual
    draw of position k where it was rejected).  p_bonus: target distribution after all drafts.
    Returns [d_1, ..., d_j, t] (length j + 1, between 1 and positions + 1)."""
    positions = len(draft)
    j = 0
    while j < positions and bool(accepted[j]):
        j += 1
    t = int(out_token[j]) if j < positions else inverse_cdf(p_bonus, u_bonus)
    return [int(d) for d in draft[:j]] + [t]


# ----------------------------------------------------------------------------------------------
# One row, all steps in the paper's order (Algorithm 1 steps 1-3 with Algorithm 4 steps 4-8)
# ----------------------------------------------------------------------------------------------
def drafter_qprime(y: np.ndarray, kappa: np.ndarray, N: int, drafter_kind: str) -> np.ndarray:
    """q = softmax(y) (or y itself when the drafter hands over probabilities), then TLI."""
    q = softmax(y) if drafter_kind == "logits" else np.asarray(y, dtype=F64)
    return tli_project(q, kappa, N)


def rdk_row(z: np.ndarray, y: np.ndarray, kappa: np.ndarray, u: np.ndarray, mode: str,
            M: np.ndarray | None = None, drafter_kind: str = "logits",
            operand_bf16: bool = False, w_given: np.ndarray | None = None,
            prior: np.ndarray | None = None) -> dict:
    """Run one row through redistribution, draft draw, rejection test and residual draw.

    z [N] target logits, y [n] drafter logits/probabilities, kappa [n] kept ids, u [trials, 4]
    uniforms (lane 0 draft, 1 accept, 2 residual).  mode: "linear" (Eq. rdk-taylor), "exact"
    (M^T q', needs M), or "given" (w_given supplied, e.g. a matrix product computed elsewhere in
    this checker).  operand_bf16 rounds q' at the kept ids to bfloat16 before the exact product
    (it is then the stored left operand of the contraction).  prior [N] (linear mode only): logits of
    the distribution that takes the place of p inside Eq. rdk-taylor (theta and w); verification is
    against p = softmax(z) all the same.  Without it the formula uses p itself (the literal reading).
    """
    z = np.asarray(z, dtype=F64)
    kappa = np.asarray(kappa, dtype=np.int64)
    N = z.size
    p = softmax(z)                                               # O1
    theta = None
    if mode == "given":
        w = np.asarray(w_given, dtype=F64)
        qp = None
    else:
        qp = drafter_qprime(y, kappa, N, drafter_kind)           # O2
        if mode == "linear":
            pi = p if prior is None else softmax(np.asarray(prior, dtype=F64))
            theta, w = redistribute_linear(pi, qp)               # O3l
        elif mode == "exact":
            valid = (kappa >= 0) & (kappa < N)
            qk = np.where(valid, qp[np.where(valid, kappa, 0)], 0.0)
            if operand_bf16:
                qk = round_to_bf16(qk)
            w = redistribute_exact(qk, M)                        # O3e
        else:
            raise ValueError(mode)
    C = np.cumsum(w)
    S = float(C[-1])                                             # O4
    qt = w / S
    alpha = acceptance_rate(p, qt)                               # O7
    R, r = residual(p, qt)                                       # O8
    Cr = np.cumsum(r)
    u = np.asarray(u, dtype=F64).reshape(-1, 4)
    T = u.shape[0]
    draft = np.zeros(T, dtype=np.int32)
    out_tok = np.zeros(T, dtype=np.int32)
    acc = np.zeros(T, dtype=bool)
    a_prob = np.zeros(T, dtype=F64)
    resid_tok = np.zeros(T, dtype=np.int32)
    for t in range(T):
        d = inverse_cdf(w, u[t, 0])                              # O5
        a, ok = accept_test(p, qt, d, u[t, 1])                   # O6
        rt = residual_sample(p, qt, u[t, 2])                     # O8 (always evaluated; used on rejection)
        draft[t], acc[t], a_prob[t], resid_tok[t] = d, ok, a, rt
        out_tok[t] = d if ok else rt
    return {"p": p, "qprime": qp, "w": w, "S": S, "qtilde": qt, "theta": theta, "alpha": alpha,
            "R": R, "r": r, "cdf_w": C, "cdf_r": Cr, "draft": draft, "accepted": acc,
            "accept_prob": a_prob, "out_token": out_tok, "residual_token": resid_tok}
