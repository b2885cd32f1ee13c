"""Pins for the CPU checker: each of its functions is tied to something other than itself --
a value worked out by hand from the paper's formulas, a closed form, a theorem's inequality, a
special case that reduces to a library routine, or brute-force enumeration on a tiny vocabulary."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import rdk_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(path):
    with open(os.path.join(GOLDEN, path)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def _rand_dist(rng, N, scale=2.0):
    z = rng.normal(0.0, scale, size=N)
    e = np.exp(z - z.max())
    return e / e.sum()


# ---------------------------------------------------------------- softmax (O1)
def test_softmax_equal_logits_uniform_and_shift_invariant():
    assert np.allclose(O.softmax(np.full(7, 3.25)), 1.0 / 7.0, rtol=0, atol=1e-16)
    rng = np.random.default_rng(0)
    z = rng.normal(0, 3, size=50)
    assert np.allclose(O.softmax(z), O.softmax(z + 123.456), rtol=1e-13, atol=0)
    assert abs(O.softmax(z).sum() - 1.0) < 1e-15
    # against the library routine
    assert np.allclose(O.softmax(z), torch.softmax(torch.from_numpy(z), 0).numpy(), rtol=1e-13)


def test_softmax_two_logits_closed_form():
    # softmax([a, b])_0 = 1 / (1 + exp(b - a))
    a, b = 0.3, -1.7
    assert abs(O.softmax(np.array([a, b]))[0] - 1.0 / (1.0 + np.exp(b - a))) < 1e-16


def test_softmax_stability_theorem_4_2():
    # ||softmax(z + eta) - softmax(z)||_1 <= 0.5 ||eta||_1
    rng = np.random.default_rng(1)
    for _ in range(200):
        m = int(rng.integers(2, 40))
        z = rng.normal(0, 3, size=m)
        eta = rng.normal(0, rng.uniform(0.01, 2.0), size=m)
        lhs = np.abs(O.softmax(z + eta) - O.softmax(z)).sum()
        assert lhs <= 0.5 * np.abs(eta).sum() + 1e-15


# ---------------------------------------------------------------- bf16 rounding
def test_round_to_bf16_matches_library_conversion():
    rng = np.random.default_rng(2)
    x32 = np.concatenate([rng.normal(0, 1, 20000), rng.normal(0, 1e-6, 20000),
                          rng.uniform(-40, 40, 20000)]).astype(np.float32)
    # ties and exact values
    x32 = np.concatenate([x32, np.array([1.0, 1.00390625, 1.01171875, 0.0, -2.5, 3.0e-39],
                                        dtype=np.float32)])
    ours = O.round_to_bf16(x32.astype(np.float64))
    lib = torch.from_numpy(x32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(ours, lib)
    # 1 + 2^-8 lies exactly between 1 and 1 + 2^-7: the even neighbour is 1
    assert O.round_to_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert O.round_to_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6


# ---------------------------------------------------------------- TLI (O2)
def test_tli_by_hand_eq_tli_drafter():
    # q over 3 kept tokens mapped to ids 4, 1, 9 (9 is outside a 5-token target vocabulary)
    q = np.array([0.2, 0.3, 0.5])
    qp = O.tli_project(q, np.array([4, 1, 9]), 5)
    assert np.allclose(qp, [0.0, 0.6, 0.0, 0.0, 0.4], atol=1e-16)
    qp = O.tli_project(q, np.array([4, 1, -1]), 5)
    assert np.allclose(qp, [0.0, 0.6, 0.0, 0.0, 0.4], atol=1e-16)
    # pruned drafter (D inside T): renormalising is a no-op
    qp = O.tli_project(q, np.array([0, 2, 3]), 5)
    assert np.allclose(qp, [0.2, 0.0, 0.3, 0.5, 0.0], atol=1e-16)


def test_tli_errors():
    with pytest.raises(O.EmptyIntersection):
        O.tli_project(np.array([1.0]), np.array([7]), 5)
    with pytest.raises(O.BadIds):
        O.tli_project(np.array([0.5, 0.5]), np.array([2, 2]), 5)


# ---------------------------------------------------------------- affinity (O0)
def test_affinity_row_stochastic_and_limits():
    rng = np.random.default_rng(3)
    N, n, d = 40, 12, 6
    E = rng.normal(size=(N, d))
    kappa = np.sort(rng.choice(N, n, replace=False))
    M = O.build_affinity(E, kappa, 0.1)
    assert M.shape == (n, N) and (M >= 0).all()
    assert np.allclose(M.sum(axis=1), 1.0, atol=1e-14)
    # tau -> infinity: every entry 1/N
    assert np.allclose(O.build_affinity(E, kappa, 1e12), 1.0 / N, atol=1e-12)
    # tau -> 0+: cos(e_i, e_i) = 1 is the strict row maximum, so M -> identity on the kept rows
    M0 = O.build_affinity(E, kappa, 1e-4)
    I = np.zeros((n, N))
    I[np.arange(n), kappa] = 1.0
    assert np.allclose(M0, I, atol=1e-12)
    # scaling an embedding does not change a cosine
    E2 = E * rng.uniform(0.1, 10.0, size=(N, 1))
    assert np.allclose(O.build_affinity(E2, kappa, 0.1), M, atol=1e-13)
    # column helper agrees with the full matrix
    cols = np.array([0, 5, 17, 39])
    assert np.allclose(O.affinity_columns(E, kappa, 0.1, cols), M[:, cols], atol=1e-16)


def test_affinity_orthonormal_closed_form():
    # orthonormal embeddings: Omega = I, so M_ii = e^{1/tau}/(e^{1/tau} + N - 1), others 1/(...)
    N, tau = 6, 0.5
    E = np.eye(N) * 3.0
    kappa = np.array([1, 4])
    M = O.build_affinity(E, kappa, tau)
    den = np.exp(1.0 / tau) + N - 1
    for r, i in enumerate(kappa):
        for j in range(N):
            want = np.exp(1.0 / tau) / den if j == i else 1.0 / den
            assert abs(M[r, j] - want) < 1e-15


def test_affinity_is_softmax_of_cosine_rows():
    # Eq. symbolic-m row by row against the library softmax of a hand-built cosine
    rng = np.random.default_rng(4)
    N, d, tau = 9, 5, 0.3
    E = rng.normal(size=(N, d))
    kappa = np.array([2, 7])
    M = O.build_affinity(E, kappa, tau)
    for r, i in enumerate(kappa):
        cos = np.array([E[i] @ E[j] / (np.linalg.norm(E[i]) * np.linalg.norm(E[j]))
                        for j in range(N)])
        want = torch.softmax(torch.from_numpy(cos / tau), 0).numpy()
        assert np.allclose(M[r], want, atol=1e-15)


def test_non_expansive_lemma():
    rng = np.random.default_rng(5)
    N = 30
    E = rng.normal(size=(N, 4))
    M = O.build_affinity(E, np.arange(N), 0.2)
    for _ in range(50):
        x, y = rng.normal(size=N), rng.normal(size=N)
        lhs = np.abs(O.redistribute_exact(x, M) - O.redistribute_exact(y, M)).sum()
        assert lhs <= np.abs(x - y).sum() + 1e-13


# ---------------------------------------------------------------- exact redistribution (O3e)
def test_exact_identity_reduces_to_tli():
    rng = np.random.default_rng(6)
    N, n = 16, 5
    kappa = np.sort(rng.choice(N, n, replace=False))
    q = _rand_dist(rng, n)
    qp = O.tli_project(q, kappa, N)
    I = np.zeros((n, N))
    I[np.arange(n), kappa] = 1.0
    w = O.redistribute_exact(qp[kappa], I)
    assert np.array_equal(w, qp)
    row = O.rdk_row(rng.normal(size=N), np.log(q), kappa, rng.uniform(size=(8, 4)), "exact", M=I)
    assert np.allclose(row["qtilde"], qp, atol=1e-15)
    assert set(row["draft"].tolist()) <= set(kappa.tolist())      # TLI never drafts OOV tokens
    assert abs(row["alpha"] - np.minimum(row["p"], qp).sum()) < 1e-15


def test_exact_m2_worked_example_theorem_4_3():
    for tok in _rows("thm43_m2_example.txt"):
        p1, p2, m11, m12, m21, m22, a_tli, a_rdk = (float(t) for t in tok)
        M = np.array([[m11, m12], [m21, m22]])
        p = np.array([p1, p2])
        qp = np.array([1.0, 0.0])
        w = O.redistribute_exact(qp, M)
        assert np.allclose(w, [m11, m12], atol=1e-16)
        assert abs(O.acceptance_rate(p, qp) - a_tli) < 1e-15
        S, qt = O.normalise(w)
        assert abs(S - 1.0) < 1e-15
        assert abs(O.acceptance_rate(p, qt) - a_rdk) < 1e-15
        assert a_tli <= O.acceptance_rate(p, qt) + 1e-15 or (p1 >= m11 and p2 < m12)


def test_exact_rectangular_by_hand_and_loops():
    # n = 2 kept rows over N = 3 tokens; w_j = sum_i q'_i M_ij
    M = np.array([[0.5, 0.25, 0.25], [0.1, 0.2, 0.7]])
    qk = np.array([0.25, 0.75])
    want = [0.25 * 0.5 + 0.75 * 0.1, 0.25 * 0.25 + 0.75 * 0.2, 0.25 * 0.25 + 0.75 * 0.7]
    assert np.allclose(O.redistribute_exact(qk, M), want, atol=1e-16)
    rng = np.random.default_rng(7)
    N, n = 16, 6
    E = rng.normal(size=(N, 5))
    kappa = np.sort(rng.choice(N, n, replace=False))
    M = O.build_affinity(E, kappa, 0.1)
    qk = _rand_dist(rng, n)
    w = O.redistribute_exact(qk, M)
    assert np.allclose(w, O.redistribute_exact_loops(qk, M), atol=1e-16)
    assert (w >= 0).all() and abs(w.sum() - 1.0) < 1e-14           # mass preserved (Assumption 4.1)


def test_theorem_4_1_bounded_l1():
    rng = np.random.default_rng(8)
    for _ in range(30):
        N = int(rng.integers(4, 30))
        n = int(rng.integers(1, N + 1))
        kappa = np.sort(rng.choice(N, n, replace=False))
        E = rng.normal(size=(N, 6))
        p = _rand_dist(rng, N)
        q0 = O.tli_project(_rand_dist(rng, n), kappa, N)
        # a full N x N row-stochastic matrix is needed for M^T p; rows of kept ids are the ones RDK uses
        Mfull = O.build_affinity(E, np.arange(N), float(rng.uniform(0.05, 1.0)))
        pprime = O.redistribute_exact(q0[kappa], Mfull[kappa])
        eps = np.abs(O.redistribute_exact(p, Mfull) - p).sum()
        assert np.abs(pprime - p).sum() <= np.abs(q0 - p).sum() + eps + 1e-13


# ---------------------------------------------------------------- linear redistribution (O3l)
def test_linear_hand_rationals_n4():
    tok = _rows("taylor_n4_rationals.txt")[0]
    vals = [Fraction(int(tok[i]), int(tok[i + 1])) for i in range(0, len(tok), 2)]
    p = np.array([0.5, 0.25, 0.125, 0.125])
    qp = np.array([0.75, 0.0, 0.25, 0.0])
    theta, w = O.redistribute_linear(p, qp)
    assert abs(theta - float(vals[0])) < 1e-16
    assert np.allclose(w, [float(v) for v in vals[1:]], rtol=1e-15, atol=0)
    # the same numbers recomputed from the formula in exact rational arithmetic
    pf = [Fraction(1, 2), Fraction(1, 4), Fraction(1, 8), Fraction(1, 8)]
    qf = [Fraction(3, 4), Fraction(0), Fraction(1, 4), Fraction(0)]
    th = sum(a * b for a, b in zip(pf, qf))
    assert th == vals[0]
    assert [(4 * b + th * a) / (4 + a) for a, b in zip(pf, qf)] == vals[1:]


def test_linear_uniform_p_closed_form():
    # p = 1/N: theta = 1/N, S = 1 exactly, q~_j = (N^3 q'_j + 1)/(N^3 + N); OOV tokens get 1/(N^3+N)
    for N, n in [(16, 4), (64, 7), (2, 1)]:
        rng = np.random.default_rng(N)
        kappa = np.sort(rng.choice(N, n, replace=False))
        qp = O.tli_project(_rand_dist(rng, n), kappa, N)
        theta, w = O.redistribute_linear(np.full(N, 1.0 / N), qp)
        S, qt = O.normalise(w)
        assert abs(theta - 1.0 / N) < 1e-16
        assert abs(S - 1.0) < 1e-14
        assert np.allclose(qt, (N ** 3 * qp + 1.0) / (N ** 3 + N), rtol=1e-13, atol=0)
        oov = np.setdiff1d(np.arange(N), kappa)
        assert np.allclose(qt[oov], 1.0 / (N ** 3 + N), rtol=1e-13, atol=0)
    assert abs(1.0 / (16 ** 3 + 16) - 2.4319e-4) < 1e-8


def test_linear_nonnegative_and_oov_mass_positive():
    rng = np.random.default_rng(9)
    N, n = 200, 20
    kappa = np.sort(rng.choice(N, n, replace=False))
    p = _rand_dist(rng, N)
    qp = O.tli_project(_rand_dist(rng, n), kappa, N)
    theta, w = O.redistribute_linear(p, qp)
    S, qt = O.normalise(w)
    oov = np.setdiff1d(np.arange(N), kappa)
    assert (w >= 0).all() and abs(qt.sum() - 1.0) < 1e-14
    assert (qt[oov] > 0).all()                                   # an OOV token can be drafted
    assert (qt[oov] < p[oov]).all()                              # and never above the target's mass
    assert abs(theta - sum(p[k] * qp[k] for k in kappa)) < 1e-16


def test_linear_tracks_exact_in_the_regime_of_theorem_4_4():
    # The proof assumes Omega_ij/tau = theta p_j (rank one) and N q'_j = 1 + O(theta): take n = N,
    # q' uniform, theta = p^T q' = 1/N.  Then ||p_Taylor - M^T q'||_1 = O(theta + 1/N^2) -> the gap
    # times N^2 stays bounded (and the gap itself vanishes) as N grows.
    rng = np.random.default_rng(10)
    gaps = []
    for N in [16, 64, 256, 1024]:
        p = _rand_dist(rng, N)
        qp = np.full(N, 1.0 / N)
        theta = float(p @ qp)
        A = np.tile(theta * p, (N, 1))                            # Omega_ij / tau
        M = np.exp(A)
        M /= M.sum(axis=1, keepdims=True)                         # Eq. symbolic-m
        exact = O.redistribute_exact(qp, M)
        th, w = O.redistribute_linear(p, qp)
        assert abs(th - theta) < 1e-16
        _, qt = O.normalise(w)
        gaps.append(np.abs(qt - exact).sum() * N * N)
    assert max(gaps) <= 2.0, gaps
    assert gaps[-1] / 1024 ** 2 < 1e-5


# ---------------------------------------------------------------- sampler (O5-O8)
def test_inverse_cdf_convention_sweep():
    w = np.array([0.0, 0.2, 0.0, 0.0, 0.5, 0.3, 0.0])
    C = np.cumsum(w)
    total = C[-1]
    assert O.inverse_cdf(w, 0.0) == 1                            # first positive-weight token
    assert O.inverse_cdf(w, 0.1) == 1
    assert O.inverse_cdf(w, 0.45) == 4
    assert O.inverse_cdf(w, 0.9) == 5
    assert O.inverse_cdf(w, np.nextafter(1.0, 0.0)) == 5          # never the trailing zero
    eps = 1e-12
    # C_j > u*total is strict: u*total == C_1 selects the NEXT positive token
    assert O.inverse_cdf(w, 0.2 / total) == 4
    assert O.inverse_cdf(w, (0.2 - eps) / total) == 1
    assert O.inverse_cdf(w, (0.7 + eps) / total) == 5
    # un-normalised weights give the same answer
    assert O.inverse_cdf(37.0 * w, 0.45) == 4
    # frequency check against the weights
    rng = np.random.default_rng(11)
    u = rng.uniform(size=20000)
    counts = np.bincount([O.inverse_cdf(w, x) for x in u], minlength=w.size)
    assert counts[[0, 2, 3, 6]].sum() == 0
    assert np.allclose(counts / u.size, w, atol=0.015)


def _enumerate_case(p, qt):
    """Exact enumeration of Algorithm 4's per-position step for a draft distribution qt."""
    N = p.size
    alpha = O.acceptance_rate(p, qt)
    R, r = O.residual(p, qt)
    acc_total = 0.0
    out = np.zeros(N)
    for d in range(N):
        if qt[d] == 0.0:
            continue
        a, _ = O.accept_test(p, qt, d, 0.5)
        acc_total += qt[d] * a
        out[d] += qt[d] * a
    if R > 0:
        out += (1.0 - acc_total) * r / R
    return alpha, R, acc_total, out


def test_sampler_exact_enumeration_small_vocab():
    rng = np.random.default_rng(12)
    for N in [2, 3, 5, 8, 16]:
        for n in sorted({1, max(1, N // 4), N}):
            for mode in ["linear", "exact"]:
                kappa = np.sort(rng.choice(N, n, replace=False))
                z, y = rng.normal(0, 2, N), rng.normal(0, 2, n)
                M = O.build_affinity(rng.normal(size=(N, 4)), kappa, 0.1)
                row = O.rdk_row(z, y, kappa, np.zeros((1, 4)), mode, M=M)
                p, qt = row["p"], row["qtilde"]
                assert abs(qt.sum() - 1.0) < 1e-14 and (qt >= 0).all()
                alpha, R, acc_total, out = _enumerate_case(p, qt)
                assert abs(acc_total - alpha) < 1e-12            # Def. 2.1: alpha = P(accept)
                assert np.allclose(out, p, atol=1e-12)           # lossless: output ~ p
                # Lemma 2.3
                k = np.maximum(0.0, qt - p)
                assert abs(alpha - (1.0 - k.sum())) < 1e-12
                assert abs(alpha - (1.0 - 0.5 * np.abs(p - qt).sum())) < 1e-12
                assert abs(R - (1.0 - alpha)) < 1e-12
                assert abs(row["alpha"] - alpha) < 1e-15 and abs(row["R"] - R) < 1e-15


def test_accept_test_cases():
    p = np.array([0.5, 0.5, 0.0])
    qt = np.array([0.25, 0.5, 0.25])
    assert O.accept_test(p, qt, 0, 0.999999) == (1.0, True)       # p >= q~: always accepted
    assert O.accept_test(p, qt, 2, 0.0) == (0.0, False)           # p = 0: never accepted
    p = np.array([0.1, 0.9])
    qt = np.array([0.4, 0.6])
    a, ok = O.accept_test(p, qt, 0, 0.24)
    assert abs(a - 0.25) < 1e-16 and ok
    assert not O.accept_test(p, qt, 0, 0.26)[1]


def test_residual_fallback_when_distributions_coincide():
    p = np.array([0.2, 0.3, 0.5])
    assert O.residual(p, p)[0] == 0.0
    assert O.residual_sample(p, p, 0.25) == 1                    # drawn from p itself
    R, r = O.residual(np.array([0.7, 0.3]), np.array([0.4, 0.6]))
    assert abs(R - 0.3) < 1e-16 and np.allclose(r, [0.3, 0.0])


def test_sampler_monte_carlo_small_vocab():
    rng = np.random.default_rng(13)
    N, n, trials = 8, 3, 120000
    kappa = np.array([1, 4, 6])
    z, y = rng.normal(0, 2, N), rng.normal(0, 2, n)
    u = rng.uniform(size=(trials, 4))
    row = O.rdk_row(z, y, kappa, u, "linear")
    alpha, p = row["alpha"], row["p"]
    freq = row["accepted"].mean()
    sigma = np.sqrt(alpha * (1 - alpha) / trials)
    assert abs(freq - alpha) < 4 * sigma
    # output histogram against p: chi-square with N - 1 degrees of freedom (99.99 % quantile ~ 29.9)
    counts = np.bincount(row["out_token"], minlength=N)
    chi2 = ((counts - trials * p) ** 2 / (trials * p)).sum()
    assert chi2 < 29.9, chi2
    # drafts follow q~ (OOV tokens included)
    dc = np.bincount(row["draft"], minlength=N)
    assert np.abs(dc / trials - row["qtilde"]).max() < 5 * np.sqrt(0.25 / trials)


def test_rdk_row_given_matches_exact_and_bf16_operand():
    rng = np.random.default_rng(14)
    N, n = 32, 8
    kappa = np.sort(rng.choice(N, n, replace=False))
    M = O.build_affinity(rng.normal(size=(N, 6)), kappa, 0.1)
    z, y, u = rng.normal(0, 2, N), rng.normal(0, 2, n), rng.uniform(size=(4, 4))
    a = O.rdk_row(z, y, kappa, u, "exact", M=M)
    b = O.rdk_row(z, None, kappa, u, "given", w_given=a["w"])
    for k in ["S", "alpha", "R"]:
        assert a[k] == b[k]
    assert np.array_equal(a["draft"], b["draft"]) and np.array_equal(a["out_token"], b["out_token"])
    c = O.rdk_row(z, y, kappa, u, "exact", M=M, operand_bf16=True)
    assert abs(c["S"] - 1.0) < 2.0 ** -8                          # rounded operand: mass nearly 1
    assert np.abs(c["qtilde"] - a["qtilde"]).max() < 2.0 ** -8
    # probabilities as drafter input give the same row as their logits
    q = O.softmax(y)
    d = O.rdk_row(z, q, kappa, u, "linear", drafter_kind="probs")
    e = O.rdk_row(z, y, kappa, u, "linear")
    assert np.allclose(d["w"], e["w"], rtol=1e-13, atol=0)


# ---------------------------------------------------------------- accepted_len (O9)
def test_accepted_len_bruteforce():
    for P in [1, 2, 3, 5]:
        pats = np.array(list(itertools.product([False, True], repeat=P)))
        got = O.accepted_len(pats)
        for row, g in zip(pats, got):
            want = 0
            for v in row:
                if not v:
                    break
                want += 1
            assert g == want
            assert g == (P if row.all() else int(np.argmin(row)))


# ---------------------------------------------------------------- emitted sequence (O10)
def test_emit_sequence_bruteforce_and_bonus_distribution():
    rng = np.random.default_rng(15)
    p_bonus = _rand_dist(rng, 6)
    for P in [1, 2, 4]:
        draft = rng.integers(0, 100, size=P)
        resid = rng.integers(100, 200, size=P)
        for pat in itertools.product([False, True], repeat=P):
            seq = O.emit_sequence(draft, pat, resid, p_bonus, 0.5)
            j = P if all(pat) else list(pat).index(False)
            assert len(seq) == j + 1 and seq[:j] == draft[:j].tolist()          # between 1 and P + 1 tokens
            if j < P:
                assert seq[-1] == resid[j]                                      # the residual draw of the first rejection
            else:
                assert seq[-1] == O.inverse_cdf(p_bonus, 0.5) and 0 <= seq[-1] < 6
    # when every draft is accepted the extra token is distributed as p
    u = rng.uniform(size=30000)
    counts = np.bincount([O.emit_sequence([7], [True], [9], p_bonus, x)[-1] for x in u], minlength=6)
    assert np.abs(counts / u.size - p_bonus).max() < 0.012


def test_linear_with_a_separate_prior():
    """Eq. rdk-taylor with a prior pi in place of p.  (i) pi = p is the literal reading, result for
    result.  (ii) A uniform prior has a closed form that does not involve the target at all:
    theta = 1/N, q~_j = (N^3 q'_j + 1) / (N^3 + N), S = 1 -- here with a non-uniform target, so the
    acceptance rate and the residual do see p.  (iii) The output token is still distributed as p."""
    rng = np.random.default_rng(12)
    N, n = 12, 5
    kappa = np.sort(rng.choice(N, n, replace=False))
    z, y = rng.normal(0, 2, N), rng.normal(0, 2, n)
    u = rng.random((3, 4))
    a = O.rdk_row(z, y, kappa, u, "linear")
    b = O.rdk_row(z, y, kappa, u, "linear", prior=z)
    for k in ("theta", "S", "alpha", "R"):
        assert a[k] == b[k]
    assert np.array_equal(a["w"], b["w"]) and np.array_equal(a["draft"], b["draft"])
    c = O.rdk_row(z, y, kappa, u, "linear", prior=np.full(N, 0.7))
    qp = c["qprime"]
    assert abs(c["theta"] - 1.0 / N) < 1e-15 and abs(c["S"] - 1.0) < 1e-12
    assert np.allclose(c["qtilde"], (N ** 3 * qp + 1.0) / (N ** 3 + N), rtol=0, atol=1e-15)
    p = O.softmax(z)
    assert abs(c["alpha"] - np.minimum(p, c["qtilde"]).sum()) < 1e-15
    # losslessness: sum_d q~_d a_d = alpha and q~_t a_t + (1 - alpha) r_t = p_t for every token t
    qt = c["qtilde"]
    acc = np.minimum(1.0, p / qt)
    r = np.maximum(0.0, p - qt)
    r = r / r.sum()
    assert abs((qt * acc).sum() - c["alpha"]) < 1e-12
    assert np.allclose(qt * acc + (1 - c["alpha"]) * r, p, rtol=0, atol=1e-12)
