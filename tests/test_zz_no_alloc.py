"""rdk_redistribute_exact_static: the exact redistribution for callers that must not allocate
device memory (for instance a serving loop that has handed all memory management to its host
framework, or code that runs while a stream is being captured).  The library stages its q' operand
in a fixed array of its own instead of a caller workspace.  The results must be those of
rdk_redistribute_exact on the same inputs; two calls in a row with different problem sizes check
that nothing left in the shared array by the first call leaks into the second."""
import ctypes as C

import pytest
import torch

import workloads as W

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


def test_static_scratch_matches_workspace_variant_twice_in_a_row():
    import paper_2506_03206_b200 as rdk
    # a larger problem first, then a smaller one with a different row length
    _case(rdk, W.tiny_config(N=2050, n=130, rows=17, trials=1, emb_dim=8, seed=21))
    _case(rdk, W.tiny_config(N=300, n=33, rows=5, trials=1, emb_dim=8, seed=22))


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
