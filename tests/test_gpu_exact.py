"""GPU parity of the affinity construction (Eq. symbolic-m), the exact redistribution w = M^T q'
(Algorithm 1 step 2) and the sampler fed with a precomputed w, against the CPU checker."""
import numpy as np
import pytest
import torch

import parity_util as PU
import workloads as W
from oracle import rdk_oracle as O

pytestmark = pytest.mark.gpu

KIND = {"logits": 0, "probs": 1}


def _rdk():
    import paper_2506_03206_b200 as rdk
    return rdk


def _oracle_M(cfg, inp):
    return O.build_affinity(W.to_f64(inp["embeddings"]), inp["kept_ids"].numpy(), cfg.tau)


def _upload_affinity(M64, layout, B):
    """Put the checker's matrix into one of the library's two layouts on the GPU."""
    n, N = M64.shape
    A = B.affinity_alloc(N, n, layout, "cuda")
    if layout == B.RDK_AFF_F32_ROWS:
        A["data"].copy_(torch.from_numpy(M64).to(torch.float32))
    else:
        A["data"][:, :n].copy_(torch.from_numpy(O.round_to_bf16(M64).T.copy()).to(torch.bfloat16))
    return A


@pytest.mark.parametrize("which", ["C1", "tiny16", "odd"])
def test_build_affinity_fp32_rows(which):
    rdk = _rdk()
    B = rdk.binding
    cfg = {"C1": W.CONFIGS["C1"], "tiny16": W.tiny_config(N=16, n=4, emb_dim=8),
           "odd": W.tiny_config(N=777, n=45, emb_dim=33, dtype="bf16")}[which]
    inp = W.make_inputs(cfg, with_embeddings=True)
    M_ref = _oracle_M(cfg, inp)
    M = rdk.rdk_build_affinity(inp["embeddings"].cuda(), inp["kept_ids"].cuda(), cfg.tau, B.RDK_AFF_F32_ROWS)
    torch.cuda.synchronize()
    got = M["data"].cpu().double().numpy()
    assert np.abs(got - M_ref).max() <= PU.ABS_TOL
    sel = M_ref > 1e-30
    assert (np.abs(got - M_ref)[sel] / M_ref[sel]).max() <= 1e-4
    assert np.abs(got.sum(axis=1) - 1.0).max() < 1e-5                 # Assumption 4.1


def test_build_affinity_bf16_cols_and_dropped_rows():
    rdk = _rdk()
    B = rdk.binding
    cfg = W.tiny_config(N=1500, n=200, emb_dim=32, dtype="bf16")
    inp = W.make_inputs(cfg, with_embeddings=True)
    ids = inp["kept_ids"].clone()
    ids[3] = -1
    ids[17] = cfg.N + 1
    M_ref = O.build_affinity(W.to_f64(inp["embeddings"]), ids.numpy(), cfg.tau)
    M = rdk.rdk_build_affinity(inp["embeddings"].cuda(), ids.cuda(), cfg.tau, B.RDK_AFF_BF16_COLS)
    torch.cuda.synchronize()
    got = M["data"][:, : cfg.n].cpu().double().numpy().T               # back to [n, N]
    # bf16 storage (8 significant bits): the stored value is the checker's value rounded to
    # nearest-even, except where the fp32 arithmetic lands on the other side of a rounding
    # boundary -- then it is the neighbouring bf16 number (one unit in the last place, 2^-7).
    M_rnd = O.round_to_bf16(M_ref)
    assert np.mean(got == M_rnd) >= 0.99
    assert np.all(np.abs(got - M_rnd) <= 2.0 ** -7 * M_rnd + 1e-38)
    assert np.all(np.abs(got - M_ref) <= (2.0 ** -8 + 1e-4) * M_ref + 1e-38)
    assert np.all(got[3] == 0) and np.all(got[17] == 0)


@pytest.mark.parametrize("N,n,d", [(3000, 300, 72), (4100, 2300, 128), (700, 64, 64)])
def test_build_affinity_on_the_tensor_cores(N, n, d):
    """bf16 embeddings of dimension >= 64 into the bf16 layout: the dot products run on the tensor cores (ragged
    embedding dimension, ragged tiles, more kept rows than one chunk, ids outside the vocabulary), compared with the
    checker's matrix rounded to bf16: equal except where fp32 arithmetic lands on the other side of a rounding
    boundary (then the neighbouring bf16 number)."""
    rdk = _rdk()
    B = rdk.binding
    cfg = W.tiny_config(N=N, n=n, emb_dim=d, dtype="bf16", seed=N + d)
    inp = W.make_inputs(cfg, with_embeddings=True)
    assert inp["embeddings"].dtype == torch.bfloat16
    ids = inp["kept_ids"].clone()
    ids[5] = -3
    ids[n - 2] = N
    M_ref = O.build_affinity(W.to_f64(inp["embeddings"]), ids.numpy(), cfg.tau)
    emb = inp["embeddings"].cuda()
    if d == 72:      # rows inside a wider buffer: a row stride of 80 elements (16-byte aligned rows)
        wide = torch.zeros(N, 80, dtype=torch.bfloat16, device="cuda")
        wide[:, :d] = emb
        emb = wide[:, :d]
        assert emb.stride(0) == 80
    M = rdk.rdk_build_affinity(emb, ids.cuda(), cfg.tau, B.RDK_AFF_BF16_COLS)
    torch.cuda.synchronize()
    got = M["data"][:, :n].cpu().double().numpy().T
    assert not np.isnan(got).any()
    M_rnd = O.round_to_bf16(M_ref)
    assert np.mean(got == M_rnd) >= 0.99
    assert np.all(np.abs(got - M_rnd) <= 2.0 ** -7 * M_rnd + 1e-38)
    assert np.all(np.abs(got - M_ref) <= (2.0 ** -8 + 1e-4) * M_ref + 1e-38)
    assert np.all(got[5] == 0) and np.all(got[n - 2] == 0)
    assert np.all(np.abs(got.sum(axis=1)[[0, 1, n - 1]] - 1.0) < 5e-3)


def _flip_allowance(qp, Mcols):
    """The left operand q' is rounded to bf16 on the GPU from an fp32 value and in the checker from a
    float64 value.  An element whose exact value lies within fp32 rounding error (2e-6 relative) of a
    bf16 rounding boundary may legitimately land on either neighbour; this returns, for each output
    column, the largest change of w such flips can cause (zero when no element is that close).
    qp: [..., n] float64 q' at the kept ids; Mcols: [n, cols]."""
    _, e = np.frexp(qp)
    ulp = np.ldexp(1.0, e - 8)
    dist_to_boundary = 0.5 * ulp - np.abs(qp - O.round_to_bf16(qp))
    near = dist_to_boundary <= 2e-6 * np.abs(qp)
    return (np.where(near, ulp, 0.0)) @ Mcols


def _exact_case(cfg, layout_name, identity=False):
    rdk = _rdk()
    B = rdk.binding
    layout = {"f32": B.RDK_AFF_F32_ROWS, "bf16": B.RDK_AFF_BF16_COLS}[layout_name]
    inp = W.make_inputs(cfg, with_embeddings=True)
    kappa = inp["kept_ids"].numpy()
    if identity:
        M64 = np.zeros((cfg.n, cfg.N))
        M64[np.arange(cfg.n), kappa] = 1.0
    else:
        M64 = _oracle_M(cfg, inp)
    if layout == B.RDK_AFF_BF16_COLS:
        M64 = O.round_to_bf16(M64)           # both sides contract the stored (rounded) matrix
    A = _upload_affinity(M64, layout, B)
    idx = rdk.rdk_prepare_ids(inp["kept_ids"].cuda(), cfg.N)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    w, S, _ = rdk.rdk_redistribute_exact(idx, inp["drafter"].cuda(), A, cfg.batch, cfg.positions,
                                         KIND[cfg.drafter_kind], status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    bf = layout == B.RDK_AFF_BF16_COLS
    w_ref = np.zeros((cfg.rows, cfg.N))
    for r in range(cfg.rows):
        ref = O.rdk_row(W.to_f64(inp["target"][r]), W.to_f64(inp["drafter"][r]), kappa, np.zeros((1, 4)), "exact",
                        M=M64, drafter_kind=cfg.drafter_kind, operand_bf16=bf)
        w_ref[r] = ref["w"]
        g = w[r].cpu().double().numpy()
        assert np.abs(g - ref["w"]).max() <= PU.ABS_TOL
        if bf:
            valid = (kappa >= 0) & (kappa < cfg.N)
            allow = _flip_allowance(np.where(valid, ref["qprime"][np.where(valid, kappa, 0)], 0.0), M64)
            assert np.all(np.abs(g - ref["w"]) <= PU.REL_TOL_BF16 * ref["w"] + allow + 1e-12)
            assert abs(float(S[r]) - ref["S"]) <= PU.ABS_TOL + allow.sum()
        else:
            if cfg.dtype == "bf16":
                assert np.all(np.abs(g - ref["w"]) <= PU.REL_TOL_BF16 * ref["w"] + 1e-12)
            assert PU.close(float(S[r]), ref["S"], False)
        if identity and not bf:
            assert np.allclose(g / g.sum(), ref["qprime"], atol=1e-6)   # M = I: RDK reduces to TLI
    # the sampler takes w as an input: both sides get the checker's w, stored as float32
    w_in = torch.from_numpy(w_ref).to(torch.float32)
    out = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_PRECOMPUTED_W, inp["target"].cuda(), None, w_in.cuda(),
                                    inp["uniforms"].cuda(), cfg.batch, cfg.positions)
    torch.cuda.synchronize()
    t = PU.compare_sampling(inp, out, range(cfg.rows), "given", w_given=w_in.double().numpy())
    PU.compare_accepted_len(out, cfg.batch, cfg.positions, cfg.trials)
    print(cfg.name, layout_name, t.summary())
    t.assert_ok(max_ambiguous_frac=0.1)
    return w_ref


def test_config1_tiny_rdk_exact():
    _exact_case(W.CONFIGS["C1"], "f32")


@pytest.mark.parametrize("N,n,rows", [(2, 1, 3), (16, 4, 5), (16, 16, 2), (300, 33, 9), (2050, 130, 17)])
def test_exact_small_shapes_fp32(N, n, rows):
    _exact_case(W.tiny_config(N=N, n=n, rows=rows, trials=8, emb_dim=8, seed=N + n), "f32")


def test_exact_identity_affinity_is_tli():
    _exact_case(W.tiny_config(N=64, n=10, rows=4, trials=8), "f32", identity=True)


def test_exact_probability_drafter_fp32():
    _exact_case(W.tiny_config(N=512, n=64, rows=4, trials=4, drafter_kind="probs", dtype="bf16", rho=0.8), "f32")


# ---------------------------------------------------------------- tensor-core layout (bf16, transposed)
@pytest.mark.parametrize("N,n,rows", [(300, 33, 9), (2050, 130, 17), (1000, 520, 300), (4096, 1024, 384),
                                      (777, 64, 129), (256, 8, 1)])
def test_exact_tensor_core_shapes(N, n, rows):
    # several 256 x 256 output tiles, ragged edges in all three dimensions, one- and two-MMA row tiles
    _exact_case(W.tiny_config(N=N, n=n, rows=rows, trials=2, emb_dim=8, seed=N + n + rows, dtype="bf16"), "bf16")


def test_exact_tensor_core_identity_affinity_is_tli():
    # M = I in bf16 is exact, so w must equal the bf16-rounded q' at the kept ids and 0 elsewhere
    rdk = _rdk()
    B = rdk.binding
    cfg = W.tiny_config(N=600, n=72, rows=5, trials=1, dtype="bf16", seed=8)
    inp = W.make_inputs(cfg)
    kappa = inp["kept_ids"].numpy()
    M64 = np.zeros((cfg.n, cfg.N))
    M64[np.arange(cfg.n), kappa] = 1.0
    A = _upload_affinity(M64, B.RDK_AFF_BF16_COLS, B)
    idx = rdk.rdk_prepare_ids(inp["kept_ids"].cuda(), cfg.N)
    w, S, _ = rdk.rdk_redistribute_exact(idx, inp["drafter"].cuda(), A, cfg.batch, cfg.positions)
    torch.cuda.synchronize()
    for r in range(cfg.rows):
        qp = O.drafter_qprime(W.to_f64(inp["drafter"][r]), kappa, cfg.N, "logits")
        g = w[r].cpu().double().numpy()
        assert np.all(g[np.setdiff1d(np.arange(cfg.N), kappa)] == 0)
        # the operand is the fp32 q' rounded to bf16; against the float64 q' that is one rounding step
        assert np.all(np.abs(g[kappa] - qp[kappa]) <= 2.0 ** -8 * qp[kappa] + 1e-12)


def test_exact_tensor_core_probability_drafter():
    _exact_case(W.tiny_config(N=1024, n=256, rows=40, trials=2, drafter_kind="probs", dtype="bf16", rho=0.8, emb_dim=16),
                "bf16")


def test_config5_full_size_sampled_outputs():
    """N = 32768, n = 8192, 1024 rows: the checker builds the whole affinity matrix (float64, rounded to
    bf16 for storage), the library contracts it on the tensor cores, and a seeded sample of output
    columns is recomputed by the checker for every row; the sampler then runs on the library's w."""
    rdk = _rdk()
    B = rdk.binding
    cfg = W.CONFIGS["C5"]
    inp = W.make_inputs(cfg, with_embeddings=True)
    kappa = inp["kept_ids"].numpy()
    E64 = W.to_f64(inp["embeddings"])
    Mt = torch.zeros(cfg.N, cfg.n, dtype=torch.bfloat16)
    rng = np.random.default_rng(5)
    cols = np.sort(rng.choice(cfg.N, 48, replace=False))
    Mcols = np.zeros((cfg.n, cols.size))
    for i0 in range(0, cfg.n, 1024):                      # the matrix in blocks of kept rows
        blk = O.round_to_bf16(O.build_affinity(E64, kappa[i0:i0 + 1024], cfg.tau))
        Mt[:, i0:i0 + 1024] = torch.from_numpy(blk.T.copy()).to(torch.bfloat16)
        Mcols[i0:i0 + 1024] = blk[:, cols]
    A = {"data": Mt.cuda(), "layout": B.RDK_AFF_BF16_COLS, "ld": cfg.n}
    idx = rdk.rdk_prepare_ids(inp["kept_ids"].cuda(), cfg.N)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    drafter = inp["drafter"].cuda()
    w, S, _ = rdk.rdk_redistribute_exact(idx, drafter, A, cfg.batch, cfg.positions, KIND[cfg.drafter_kind],
                                         status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # sampled columns of every row against the checker (operand rounded to bf16 as in the library)
    q = W.to_f64(inp["drafter"])
    qp64 = q / q.sum(axis=1, keepdims=True)
    ref = O.round_to_bf16(qp64) @ Mcols
    got = w[:, torch.from_numpy(cols).cuda()].cpu().double().numpy()
    assert np.all(np.abs(got - ref) <= PU.REL_TOL_BF16 * ref + _flip_allowance(qp64, Mcols) + 1e-12)
    assert np.abs(got - ref).max() <= PU.ABS_TOL
    assert torch.all((S - 1).abs() < 5e-3)                # bf16 rows of M sum to 1 only approximately
    # the library's own affinity construction at this size, on the same sampled columns
    Mg = rdk.rdk_build_affinity(inp["embeddings"].cuda(), inp["kept_ids"].cuda(), cfg.tau, B.RDK_AFF_BF16_COLS)
    torch.cuda.synchronize()
    got_cols = Mg["data"][torch.from_numpy(cols).cuda(), : cfg.n].cpu().double().numpy().T
    assert np.mean(got_cols == Mcols) >= 0.99
    assert np.all(np.abs(got_cols - Mcols) <= 2.0 ** -7 * Mcols + 1e-38)
    # sampler (precomputed-w mode) at full size: its w input is the checker's product for a sample of
    # rows (float32), placed in the rows the checker recomputes; the other rows keep the library's w
    rows = sorted(set([0, cfg.rows - 1] + rng.choice(cfg.rows, 10, replace=False).tolist()))
    w_rows = torch.from_numpy(O.round_to_bf16(qp64[rows]) @ np.vstack([O.round_to_bf16(O.build_affinity(E64, kappa[i0:i0 + 1024], cfg.tau))
                                                                      for i0 in range(0, cfg.n, 1024)])).to(torch.float32)
    w[torch.tensor(rows).cuda()] = w_rows.cuda()
    out = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_PRECOMPUTED_W, inp["target"].cuda(), None, w, inp["uniforms"].cuda(),
                                    cfg.batch, cfg.positions)
    torch.cuda.synchronize()
    t = PU.compare_sampling(inp, out, rows, "given", w_given=w_rows.double().numpy())
    print("C5", t.summary())
    t.assert_ok(max_ambiguous_frac=0.2)
