"""GPU parity of rdk_emit_sequences (Algorithm 4 steps 7-9) against the CPU checker."""
import numpy as np
import pytest
import torch

import parity_util as PU
import workloads as W
from oracle import rdk_oracle as O

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("N,positions,dtype", [(50, 3, "f32"), (5000, 5, "bf16"), (20000, 2, "bf16"), (1, 1, "f32")])
def test_emit_sequences(N, positions, dtype):
    import paper_2506_03206_b200 as rdk
    batch, trials = 12, 4
    rng = np.random.default_rng(N + positions)
    cfg = W.tiny_config(N=N, n=1, rows=batch, dtype=dtype, trials=trials, seed=N)
    bonus = W.make_inputs(cfg)["target"]                                  # [batch, N] logits
    u = torch.from_numpy(W.uniforms(N * 7 + 1, batch * positions, trials))
    # the entry point is a pure function of its inputs: any accept pattern will do, all-accepted included
    acc = rng.uniform(size=(batch, positions, trials)) < 0.7
    acc[0] = True
    acc[1] = False
    draft = rng.integers(0, N, size=(batch, positions, trials)).astype(np.int32)
    resid = rng.integers(0, N, size=(batch, positions, trials)).astype(np.int32)
    seq, ln = rdk.rdk_emit_sequences(N, batch, positions, bonus.cuda(), u.cuda(),
                                     torch.from_numpy(draft).cuda(), torch.from_numpy(acc.astype(np.uint8)).cuda(),
                                     torch.from_numpy(resid).cuda())
    torch.cuda.synchronize()
    seq, ln = seq.cpu().numpy(), ln.cpu().numpy()
    un = u.numpy().reshape(batch, positions, trials, 4)
    ambiguous = 0
    for b in range(batch):
        p = O.softmax(W.to_f64(bonus[b]))
        cdf = np.cumsum(p)
        for t in range(trials):
            ub = float(un[b, positions - 1, t, 3])
            want = O.emit_sequence(draft[b, :, t], acc[b, :, t], resid[b, :, t], p, ub)
            assert ln[b, t] == len(want)
            got = seq[b, t, : ln[b, t]].tolist()
            assert got[:-1] == want[:-1]
            if got[-1] != want[-1]:
                assert len(want) == positions + 1                          # only the bonus draw is a float decision
                assert PU.interval_distance(cdf, got[-1], ub * cdf[-1]) <= PU.BOUNDARY_TOL and p[got[-1]] > 0
                ambiguous += 1
            assert np.all(seq[b, t, ln[b, t]:] == -1)                      # entries beyond the length are untouched
    assert ambiguous <= 1
