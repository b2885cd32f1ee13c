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
        if bf or cfg.dtype == "bf16":
            assert np.all(np.abs(g - ref["w"]) <= PU.REL_TOL_BF16 * ref["w"] + 1e-12)
        assert PU.close(float(S[r]), ref["S"], bf)
        if identity and not bf:
            assert np.allclose(g / g.sum(), ref["qprime"], atol=1e-6)   # M = I: RDK reduces to TLI
    out = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_PRECOMPUTED_W, inp["target"].cuda(), None, w, inp["uniforms"].cuda(),
                                    cfg.batch, cfg.positions)
    torch.cuda.synchronize()
    # the sampler is checked on the w it was given (the GPU's own w widened exactly to float64)
    t = PU.compare_sampling(inp, out, range(cfg.rows), "given", w_given=w.cpu().double().numpy())
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
