"""rdk_redistribute_exact_static: the exact redistribution for callers that must not allocate
device memory (for instance a serving loop that has handed all memory management to its host
framework, or code that runs while a stream is being captured).  The library stages its q' operand
in a fixed array of its own instead of a caller workspace.  The results must be those of
rdk_redistribute_exact on the same inputs; two calls in a row with different problem sizes check
that nothing left in the shared array by the first call leaks into the second."""
import ctypes as C

import numpy as np
import pytest
import torch

import parity_util as PU
import workloads as W
from oracle import rdk_oracle as O

pytestmark = pytest.mark.gpu


def _case(rdk, cfg):
    B = rdk.binding
    inp = W.make_inputs(cfg, with_embeddings=True)
    kid = inp["kept_ids"].cuda()
    idx = rdk.rdk_prepare_ids(kid, cfg.N)
    M = rdk.rdk_build_affinity(inp["embeddings"].cuda(), kid, cfg.tau, B.RDK_AFF_F32_ROWS)
    drafter = inp["drafter"].cuda()
    w_ref, S_ref, _ = rdk.rdk_redistribute_exact(idx, drafter, M, cfg.batch, cfg.positions)
    w = torch.full((cfg.rows, cfg.N), float("nan"), dtype=torch.float32, device="cuda")
    S = torch.full((cfg.rows,), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rdk.rdk_redistribute_exact_static(idx, drafter, M, cfg.batch, cfg.positions, w, S, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert (w - w_ref).abs().max().item() <= 1e-5          # the tolerance of the other fp32 parity tests
    assert (S - S_ref).abs().max().item() <= 1e-5
    assert torch.all((S - 1).abs() < 1e-4)
    # and against the CPU checker: w = M^T q' with the checker's own matrix
    M64 = O.build_affinity(W.to_f64(inp["embeddings"]), inp["kept_ids"].numpy(), cfg.tau)
    kappa = inp["kept_ids"].numpy()
    for r in range(cfg.rows):
        ref = O.rdk_row(W.to_f64(inp["target"][r]), W.to_f64(inp["drafter"][r]), kappa, np.zeros((1, 4)), "exact", M=M64)
        assert np.abs(w[r].cpu().double().numpy() - ref["w"]).max() <= PU.ABS_TOL
        assert abs(float(S[r]) - ref["S"]) <= PU.ABS_TOL


def _case_tensor_cores(rdk, cfg):
    """The bf16 layout: the q' operand in the library's own array is read by the tensor-core kernel's bulk
    tensor copies.  Compared with the workspace variant (bit for bit: same kernel, same operand) and with
    the checker's product of the bf16-rounded operands."""
    from test_gpu_exact import _flip_allowance
    B = rdk.binding
    inp = W.make_inputs(cfg, with_embeddings=True)
    kid = inp["kept_ids"].cuda()
    idx = rdk.rdk_prepare_ids(kid, cfg.N)
    M64 = O.build_affinity(W.to_f64(inp["embeddings"]), inp["kept_ids"].numpy(), cfg.tau)
    A = B.affinity_alloc(cfg.N, cfg.n, B.RDK_AFF_BF16_COLS, "cuda")
    A["data"][:, : cfg.n].copy_(torch.from_numpy(O.round_to_bf16(M64).T.copy()).to(torch.bfloat16))
    drafter = inp["drafter"].cuda()
    w_ref, S_ref, _ = rdk.rdk_redistribute_exact(idx, drafter, A, cfg.batch, cfg.positions)
    w = torch.full((cfg.rows, cfg.N), float("nan"), dtype=torch.float32, device="cuda")
    S = torch.full((cfg.rows,), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rdk.rdk_redistribute_exact_static(idx, drafter, A, cfg.batch, cfg.positions, w, S, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(w, w_ref)
    assert (S - S_ref).abs().max().item() <= 1e-5          # row sums are accumulated by atomics: order may differ
    kappa = inp["kept_ids"].numpy()
    Mr = O.round_to_bf16(M64)
    qp = np.stack([O.drafter_qprime(W.to_f64(inp["drafter"][r]), kappa, cfg.N, cfg.drafter_kind)[kappa] for r in range(cfg.rows)])
    ref = O.round_to_bf16(qp) @ Mr
    got = w.cpu().double().numpy()
    assert np.all(np.abs(got - ref) <= PU.REL_TOL_BF16 * ref + _flip_allowance(qp, Mr) + 1e-12)
    assert np.abs(got - ref).max() <= PU.ABS_TOL


def test_static_scratch_matches_workspace_variant_twice_in_a_row():
    import paper_2506_03206_b200 as rdk
    # a larger problem first, then a smaller one with a different row length
    _case(rdk, W.tiny_config(N=2050, n=130, rows=17, trials=1, emb_dim=8, seed=21))
    _case(rdk, W.tiny_config(N=300, n=33, rows=5, trials=1, emb_dim=8, seed=22))


def test_static_scratch_feeds_the_tensor_core_kernel_twice_in_a_row():
    import paper_2506_03206_b200 as rdk
    _case_tensor_cores(rdk, W.tiny_config(N=2050, n=130, rows=17, trials=1, emb_dim=8, seed=23, dtype="bf16"))
    _case_tensor_cores(rdk, W.tiny_config(N=520, n=72, rows=9, trials=1, emb_dim=8, seed=24, dtype="bf16"))


def test_static_scratch_rejects_oversized_problems():
    import paper_2506_03206_b200 as rdk
    B = rdk.binding
    L = B.lib()
    pb = B.rdk_problem()
    pb.N, pb.n, pb.batch, pb.positions = 4096, 2048, 1024, 1      # operand: 1024 x 2048 floats = 8 MiB
    aff = B.rdk_affinity()
    aff.layout, aff.ld, aff.data = B.RDK_AFF_F32_ROWS, 4096, 256
    dummy = C.c_void_p(256)
    st = L.rdk_redistribute_exact_static(C.byref(pb), dummy, C.byref(aff), dummy, None, None, None)
    assert st == B.RDK_ERR_WORKSPACE_TOO_SMALL
    assert b"scratch" in L.rdk_last_error()
    assert L.rdk_exact_workspace_bytes(C.byref(pb), B.RDK_AFF_F32_ROWS) > B.RDK_STATIC_SCRATCH_BYTES
