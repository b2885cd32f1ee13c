"""Host-side checks of the seeded input generators."""
import os

import numpy as np
import torch

import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_philox_known_answers():
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for tok in rows:
        v = np.array([int(t, 16) for t in tok], dtype=np.uint32)
        assert np.array_equal(W.philox4x32_10(v[:4], v[4:6]), v[6:])


def test_uniforms_range_and_determinism():
    u = W.uniforms(42, 50, 16)
    assert u.shape == (50, 16, 4) and u.dtype == np.float32
    assert (u >= 0).all() and (u < 1).all()
    assert np.array_equal(u, W.uniforms(42, 50, 16))
    assert not np.array_equal(u, W.uniforms(43, 50, 16))
    assert abs(u.mean() - 0.5) < 0.02
    # exactly representable 24-bit fractions
    assert np.array_equal(u * 2 ** 24, np.round(u * 2 ** 24))


def test_config_shapes_match_the_named_workloads():
    c = W.CONFIGS
    assert (c["C1"].N, c["C1"].n, c["C1"].rows, c["C1"].trials) == (1024, 256, 4, 16)
    assert (c["C2"].N, c["C2"].n, c["C2"].rows) == (128256, 32064, 320)
    assert (c["C3"].N, c["C3"].n, c["C3"].rows) == (128256, 12826, 2048)
    assert (c["C4"].N, c["C4"].n, c["C4"].rows) == (262144, 32768, 2048)
    assert (c["C5"].N, c["C5"].n, c["C5"].rows) == (32768, 8192, 1024)


def test_kept_ids_rules():
    cfg = W.tiny_config(N=1000, n=100, kept_rule="zipf")
    ids = W.kept_ids(cfg)
    assert ids.dtype == torch.int32 and ids.numel() == 100
    assert torch.all(ids[1:] > ids[:-1])
    ranks = W.token_ranks(cfg)
    assert sorted(ranks[ids.long()].tolist()) == list(range(1, 101))   # the 100 most frequent
    ids_u = W.kept_ids(W.tiny_config(N=1000, n=100, kept_rule="uniform"))
    assert torch.all(ids_u[1:] > ids_u[:-1]) and ids_u.max() < 1000 and ids_u.min() >= 0


def test_make_inputs_small():
    cfg = W.tiny_config(N=512, n=64, rows=6, dtype="bf16", trials=2, rho=0.8, kept_rule="zipf",
                        zipf_bias=True)
    a = W.make_inputs(cfg)
    b = W.make_inputs(cfg)
    assert a["target"].shape == (6, 512) and a["target"].dtype == torch.bfloat16
    assert a["drafter"].shape == (6, 64) and a["uniforms"].shape == (6, 2, 4)
    assert torch.equal(a["target"], b["target"]) and torch.equal(a["drafter"], b["drafter"])
    c = W.make_inputs(cfg, variant=1)
    assert not torch.equal(a["target"], c["target"])
    # correlated component: drafter noise follows the target noise on the kept ids
    big = W.make_inputs(W.tiny_config(N=4096, n=1024, rows=8, rho=0.8))
    z = big["target"][:, big["kept_ids"].long()].flatten().double()
    y = big["drafter"].flatten().double()
    assert abs(torch.corrcoef(torch.stack([z, y]))[0, 1].item() - 0.8) < 0.05


def test_probs_drafter_is_a_distribution():
    cfg = W.tiny_config(N=256, n=32, rows=4, dtype="bf16", drafter_kind="probs", rho=0.8)
    a = W.make_inputs(cfg)
    s = a["drafter"].double().sum(dim=1)
    assert torch.all((s - 1).abs() < 2e-2) and torch.all(a["drafter"].double() >= 0)
