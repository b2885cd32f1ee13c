"""GPU parity of the linear-time path (Eq. rdk-taylor + Algorithm 4 steps 4-8) against the CPU
checker, through the C ABI, on the same seeded inputs and the same Philox uniforms."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import rdk_oracle as O
import parity_util as PU

pytestmark = pytest.mark.gpu

KIND = {"logits": 0, "probs": 1}


def _rdk():
    import paper_2506_03206_b200 as rdk
    return rdk


def _run_linear(cfg, inp, rows=None, check_qtilde=True, kept_override=None):
    rdk = _rdk()
    B = rdk.binding
    dev = "cuda"
    kid = (kept_override if kept_override is not None else inp["kept_ids"]).to(dev)
    idx = rdk.rdk_prepare_ids(kid, cfg.N)
    target, drafter, uni = inp["target"].to(dev), inp["drafter"].to(dev), inp["uniforms"].to(dev)
    kind = KIND[cfg.drafter_kind]
    out = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_LINEAR, target, drafter, None, uni, cfg.batch,
                                    cfg.positions, kind)
    torch.cuda.synchronize()
    B.check_status_word(out)
    rows = list(range(cfg.rows)) if rows is None else rows
    kappa = kid.cpu().numpy()
    tally = PU.compare_sampling(inp, out, rows, "linear", kept_ids=kappa)
    PU.compare_accepted_len(out, cfg.batch, cfg.positions, cfg.trials)
    if check_qtilde:
        qt, theta, S = rdk.rdk_redistribute_linear(idx, target, drafter, cfg.batch, cfg.positions, kind)
        torch.cuda.synchronize()
        refs = {}
        for r in rows:
            refs[r] = O.rdk_row(W.to_f64(inp["target"][r]), W.to_f64(inp["drafter"][r]), kappa,
                                np.zeros((1, 4)), "linear", drafter_kind=cfg.drafter_kind)
            assert PU.close(float(theta[r]), refs[r]["theta"], cfg.dtype == "bf16")
            assert PU.close(float(S[r]), refs[r]["S"], cfg.dtype == "bf16")
        PU.compare_qtilde(qt, refs, cfg.dtype == "bf16")
    tally.record(cfg.name)
    return tally


def test_config1_tiny_rdk_linear():
    cfg = W.CONFIGS["C1"]
    _run_linear(cfg, W.make_inputs(cfg)).assert_ok()


@pytest.mark.parametrize("N,n", [(2, 1), (2, 2), (16, 1), (16, 4), (16, 16), (17, 5), (1000, 77),
                                 (4096, 512), (4097, 1), (12289, 3000)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_small_shapes_linear(N, n, dtype):
    cfg = W.tiny_config(N=N, n=n, rows=5, dtype=dtype, trials=16, seed=N * 31 + n)
    _run_linear(cfg, W.make_inputs(cfg)).assert_ok(max_ambiguous_frac=0.1)


def test_probability_drafter_linear():
    cfg = W.tiny_config(N=3000, n=700, rows=4, dtype="bf16", trials=8, drafter_kind="probs", rho=0.8)
    _run_linear(cfg, W.make_inputs(cfg)).assert_ok()
    cfg = W.tiny_config(N=515, n=100, rows=3, dtype="f32", trials=8, drafter_kind="probs", rho=0.8)
    _run_linear(cfg, W.make_inputs(cfg)).assert_ok()


def test_zipf_pruned_mid_size_spans_several_tiles():
    # several 4096-token tiles plus a ragged tail, Zipf-ranked kept ids, correlated logits
    cfg = W.tiny_config(N=3 * 4096 + 1032, n=3300, rows=6, dtype="bf16", trials=4, kept_rule="zipf",
                        zipf_bias=True, rho=0.8, seed=11)
    _run_linear(cfg, W.make_inputs(cfg)).assert_ok()


def test_unsorted_and_out_of_vocabulary_ids():
    cfg = W.tiny_config(N=2000, n=300, rows=4, dtype="f32", trials=8, seed=5)
    inp = W.make_inputs(cfg)
    g = torch.Generator().manual_seed(3)
    ids = inp["kept_ids"][torch.randperm(cfg.n, generator=g)].clone()    # any order is accepted
    ids[7] = -1                                                          # drafter tokens outside T
    ids[100] = cfg.N + 5
    ids[299] = cfg.N
    t = _run_linear(cfg, inp, kept_override=ids)
    t.assert_ok()


def test_strided_rows_and_unaligned_rows():
    rdk = _rdk()
    B = rdk.binding
    cfg = W.tiny_config(N=1001, n=99, rows=4, dtype="bf16", trials=4, seed=9)   # odd N: rows not 16-byte aligned
    _run_linear(cfg, W.make_inputs(cfg)).assert_ok()
    # rows embedded in a wider buffer (row stride > N)
    inp = W.make_inputs(cfg)
    wide = torch.zeros(cfg.rows, cfg.N + 23, dtype=torch.bfloat16)
    wide[:, : cfg.N] = inp["target"]
    idx = rdk.rdk_prepare_ids(inp["kept_ids"].cuda(), cfg.N)
    tgt = wide.cuda()[:, : cfg.N]
    out = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_LINEAR, tgt, inp["drafter"].cuda(), None,
                                    inp["uniforms"].cuda(), cfg.batch, cfg.positions)
    torch.cuda.synchronize()
    PU.compare_sampling(inp, out, range(cfg.rows), "linear").assert_ok()


def test_directed_out_of_vocabulary_draw():
    # Aim the draft uniform into the CDF interval of a pruned token: the sampler must return it.
    rdk = _rdk()
    B = rdk.binding
    for N, n in [(16, 4), (64, 8)]:
        cfg = W.tiny_config(N=N, n=n, rows=6, dtype="f32", trials=4, seed=N)
        inp = W.make_inputs(cfg)
        kappa = inp["kept_ids"].numpy()
        oov = np.setdiff1d(np.arange(N), kappa)
        u = inp["uniforms"].clone()
        wanted = []
        for r in range(cfg.rows):
            ref = O.rdk_row(W.to_f64(inp["target"][r]), W.to_f64(inp["drafter"][r]), kappa, np.zeros((1, 4)), "linear")
            j = int(oov[np.argmax(ref["w"][oov])])
            lo = ref["cdf_w"][j - 1] if j else 0.0
            mid = 0.5 * (lo + ref["cdf_w"][j]) / ref["S"]
            u[r, :, 0] = float(np.float32(mid))
            wanted.append(j)
        inp["uniforms"] = u
        idx = rdk.rdk_prepare_ids(inp["kept_ids"].cuda(), N)
        out = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_LINEAR, inp["target"].cuda(), inp["drafter"].cuda(),
                                        None, u.cuda(), cfg.batch, cfg.positions)
        torch.cuda.synchronize()
        t = PU.compare_sampling(inp, out, range(cfg.rows), "linear")
        t.assert_ok()
        d = out["draft_token"].cpu().numpy().reshape(cfg.rows, cfg.trials)
        hits = sum(int(d[r, 0] == wanted[r]) for r in range(cfg.rows))
        assert hits >= cfg.rows - 1 and all(w not in kappa for w in wanted)


def test_identical_distributions_fall_back_to_p_for_the_residual():
    # N = 1: q~ = p = [1]; the residual mass is 0, every draft is accepted with probability 1
    rdk = _rdk()
    B = rdk.binding
    cfg = W.tiny_config(N=1, n=1, rows=2, dtype="f32", trials=4)
    inp = W.make_inputs(cfg)
    inp["kept_ids"] = torch.zeros(1, dtype=torch.int32)
    idx = rdk.rdk_prepare_ids(inp["kept_ids"].cuda(), 1)
    out = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_LINEAR, inp["target"].cuda(), inp["drafter"].cuda(), None,
                                    inp["uniforms"].cuda(), cfg.batch, cfg.positions)
    torch.cuda.synchronize()
    assert torch.all(out["draft_token"] == 0) and torch.all(out["out_token"] == 0)
    assert torch.all(out["accepted"] == 1)
    assert torch.allclose(out["alpha"].cpu(), torch.ones(2), atol=1e-6)


def test_groups_of_three_and_two_ctas():
    # 40000 bf16 logits -> three CTAs share a row; 12000 fp32 logits -> two
    cfg = W.tiny_config(N=40000, n=9000, rows=5, dtype="bf16", trials=4, kept_rule="zipf", zipf_bias=True,
                        rho=0.7, seed=41)
    _run_linear(cfg, W.make_inputs(cfg), check_qtilde=False).assert_ok()
    cfg = W.tiny_config(N=12000, n=1500, rows=5, dtype="f32", trials=16, rho=0.5, seed=42)
    _run_linear(cfg, W.make_inputs(cfg), check_qtilde=False).assert_ok()


def test_kept_ids_crowded_into_one_slice():
    # every kept id lies in the first part of the vocabulary: the kept-token caches of the first warps
    # overflow and the rest of their kept tokens take the uncached route
    cfg = W.tiny_config(N=70000, n=6000, rows=4, dtype="bf16", trials=8, rho=0.8, seed=43)
    inp = W.make_inputs(cfg)
    ids = torch.arange(cfg.n, dtype=torch.int32) + 100
    _run_linear(cfg, inp, kept_override=ids, check_qtilde=False).assert_ok()
    # the same ids in a scrambled order (rank -> drafter index table in use: generic row kernel)
    g = torch.Generator().manual_seed(4)
    _run_linear(cfg, inp, kept_override=ids[torch.randperm(cfg.n, generator=g)], check_qtilde=False).assert_ok()


def test_stream_kernel_probs_and_full_vocab():
    # n = N (nothing pruned) and a probability drafter through the streaming kernels
    cfg = W.tiny_config(N=8192, n=8192, rows=3, dtype="bf16", trials=8, rho=0.9, seed=44)
    _run_linear(cfg, W.make_inputs(cfg), check_qtilde=False).assert_ok()
    cfg = W.tiny_config(N=20000, n=4000, rows=3, dtype="bf16", trials=8, drafter_kind="probs", rho=0.8, seed=45)
    _run_linear(cfg, W.make_inputs(cfg), check_qtilde=False).assert_ok()


def test_many_rows_per_group_every_row_checked():
    """A group of three CTAs takes some thirty rows in turn: stages, live-row buffers and barrier
    phases all wrap several times.  Every row is compared with the checker."""
    cfg = W.tiny_config(N=40000, n=7000, rows=1500, dtype="bf16", trials=1, kept_rule="zipf", zipf_bias=True,
                        rho=0.8, seed=51)
    _run_linear(cfg, W.make_inputs(cfg), check_qtilde=False).assert_ok()


def test_drafter_values_far_below_their_neighbours():
    """The streaming kernels scale a warp's exponentials by the first value of the warp's range (kept
    drafter values, target logits) and fall back to the maximum when that value lies far below it: make
    many such values very small (and some -inf) so that both routes run."""
    cfg = W.tiny_config(N=30000, n=6000, rows=6, dtype="bf16", trials=4, kept_rule="zipf", zipf_bias=True,
                        rho=0.8, seed=61)
    inp = W.make_inputs(cfg)
    y = inp["drafter"].clone()
    y[:, ::7] = -250.0
    y[:, 5::31] = float("-inf")
    inp["drafter"] = y
    _run_linear(cfg, inp, check_qtilde=False).assert_ok()
    # the same for the target logits, whose scale is the first logit of each 1024-token segment
    z = inp["target"].clone()
    z[:, ::1024] = -300.0
    z[:, 2048] = float("-inf")
    z[:, 5000:5003] = float("-inf")
    inp["target"] = z
    _run_linear(cfg, inp, check_qtilde=False).assert_ok()


def test_vocabulary_beyond_sixteen_full_groups():
    # N = 300000: segments of five vectors per lane (the generic sweep), fifteen CTAs per row
    cfg = W.tiny_config(N=300000, n=2500, rows=3, dtype="bf16", trials=4, kept_rule="zipf", zipf_bias=True,
                        rho=0.8, seed=71)
    assert _rdk().rdk_stream_geometry(cfg.N, cfg.n)["segment_tokens"] == 1280
    _run_linear(cfg, W.make_inputs(cfg), check_qtilde=False).assert_ok()


def test_few_rows_fewer_than_the_pipeline_depth():
    # one and two rows: the deferred second visits all happen after the row loop
    for rows in (1, 2):
        cfg = W.tiny_config(N=20000, n=3000, rows=rows, dtype="bf16", trials=8, rho=0.6, seed=52 + rows)
        _run_linear(cfg, W.make_inputs(cfg), check_qtilde=False).assert_ok()


def test_calls_back_to_back_share_one_workspace():
    """Five calls queued on one stream with no synchronisation between them, all on the same workspace
    but each with its own inputs and outputs: a call's first kernel may start while the previous call's
    second kernel is still reading the workspace, and must not disturb it."""
    rdk = _rdk()
    B = rdk.binding
    cfgs = [W.tiny_config(N=36000, n=7000, rows=60, dtype="bf16", trials=2, kept_rule="zipf", zipf_bias=True,
                          rho=0.8, seed=80 + i) for i in range(5)]
    inps = [W.make_inputs(c) for c in cfgs]
    kid = inps[0]["kept_ids"].to("cuda")          # one kept set for all five calls
    idx = rdk.rdk_prepare_ids(kid, cfgs[0].N)
    dev = [{k: inp[k].to("cuda") for k in ("target", "drafter", "uniforms")} for inp in inps]
    ws = None
    outs = []
    torch.cuda.synchronize()
    for c, d in zip(cfgs, dev):
        o = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_LINEAR, d["target"], d["drafter"], None, d["uniforms"],
                                      c.batch, c.positions, 0, ws=ws)
        ws = o["_ws"]
        outs.append(o)
    torch.cuda.synchronize()
    for c, inp, o in zip(cfgs, inps, outs):
        B.check_status_word(o)
        PU.compare_sampling(inp, o, range(c.rows), "linear", kept_ids=kid.cpu().numpy()).assert_ok()
        PU.compare_accepted_len(o, c.batch, c.positions, c.trials)


def test_replayed_graph_with_new_inputs_in_the_same_buffers():
    """One call captured in a CUDA graph and replayed four times, each time with new logits and uniforms
    copied into the same device buffers: the host's part of the call is frozen in the graph, so whatever
    tells one launch's records in the workspace from the previous launch's must live on the device."""
    rdk = _rdk()
    B = rdk.binding
    cfgs = [W.tiny_config(N=36000, n=7000, rows=60, dtype="bf16", trials=2, kept_rule="zipf", zipf_bias=True,
                          rho=0.8, seed=90 + i) for i in range(4)]
    inps = [W.make_inputs(c) for c in cfgs]
    c0 = cfgs[0]
    kid = inps[0]["kept_ids"].to("cuda")          # one kept set for all replays
    idx = rdk.rdk_prepare_ids(kid, c0.N)
    buf = {k: inps[0][k].to("cuda").clone() for k in ("target", "drafter", "uniforms")}
    # a first call outside the capture (one-time set-up of the kernels), then the captured one
    out = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_LINEAR, buf["target"], buf["drafter"], None, buf["uniforms"],
                                    c0.batch, c0.positions, 0)
    ws = out["_ws"]
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        rdk.rdk_sample_and_verify(idx, B.RDK_MODE_LINEAR, buf["target"], buf["drafter"], None, buf["uniforms"],
                                  c0.batch, c0.positions, 0, out=out, ws=ws)
    for c, inp in zip(cfgs, inps):
        for k in buf:
            buf[k].copy_(inp[k])
        graph.replay()
        torch.cuda.synchronize()
        B.check_status_word(out)
        got = {k: v.clone() for k, v in out.items() if v is not None and k != "_ws"}
        PU.compare_sampling(inp, got, range(c.rows), "linear", kept_ids=kid.cpu().numpy()).assert_ok()
        PU.compare_accepted_len(got, c.batch, c.positions, c.trials)


def test_inputs_written_by_the_kernel_queued_just_before_the_call():
    """The logits of a call are usually the output of the kernel queued right before it.  The streaming
    kernel is launched so that it may start while that kernel drains; it must not read its inputs before
    that kernel is complete.  Thirty calls, each preceded on the same stream (no synchronisation) by
    kernels that overwrite the same input buffers with new rows; every call is checked against the checker."""
    rdk = _rdk()
    B = rdk.binding
    cfgs = [W.tiny_config(N=36000, n=7000, rows=48, dtype="bf16", trials=1, kept_rule="zipf", zipf_bias=True,
                          rho=0.8, seed=300 + i) for i in range(30)]
    inps = [W.make_inputs(c) for c in cfgs]
    c0 = cfgs[0]
    kid = inps[0]["kept_ids"].to("cuda")          # one kept set for all calls
    idx = rdk.rdk_prepare_ids(kid, c0.N)
    src = [{k: inp[k].to("cuda") for k in ("target", "drafter", "uniforms")} for inp in inps]
    buf = {k: torch.empty_like(v) for k, v in src[0].items()}
    outs, ws = [], None
    torch.cuda.synchronize()
    for s_ in src:
        for k in buf:
            buf[k].copy_(s_[k])                    # device-to-device copy kernels: the producers
        o = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_LINEAR, buf["target"], buf["drafter"], None, buf["uniforms"],
                                      c0.batch, c0.positions, 0, ws=ws)
        ws = o["_ws"]
        outs.append(o)
    torch.cuda.synchronize()
    tally = PU.Tally()
    for c, inp, o in zip(cfgs, inps, outs):
        B.check_status_word(o)
        PU.compare_sampling(inp, o, range(c.rows), "linear", tally=tally, kept_ids=kid.cpu().numpy())
    tally.record("producer_before_call")
    tally.assert_ok()


def test_a_wait_that_runs_out_reports_a_timeout_and_leaves_the_device_usable():
    """Failure path without a fault or a hang: with the spin limit of the device-side waits set to one
    failed try, the waits of an ordinary call run out (the row scalars that the CTAs of a group exchange
    are never there on the first try), every warp still reaches the end of the kernel, and the status
    word says RDK_ERR_TIMEOUT.  With the default limit restored the same call is correct again."""
    rdk = _rdk()
    B = rdk.binding
    cfg = W.tiny_config(N=40000, n=7000, rows=64, dtype="bf16", trials=1, kept_rule="zipf", zipf_bias=True,
                        rho=0.8, seed=77)
    inp = W.make_inputs(cfg)
    kid = inp["kept_ids"].cuda()
    idx = rdk.rdk_prepare_ids(kid, cfg.N)
    dev = {k: inp[k].cuda() for k in ("target", "drafter", "uniforms")}
    try:
        rdk.rdk_test_set_spin_limit(1)
        out = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_LINEAR, dev["target"], dev["drafter"], None, dev["uniforms"],
                                        cfg.batch, cfg.positions)
        torch.cuda.synchronize()
        assert int(out["status_word"].item()) == B.RDK_ERR_TIMEOUT
        with pytest.raises(B.RdkError):
            B.check_status_word(out)
    finally:
        rdk.rdk_test_set_spin_limit(0)
    out = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_LINEAR, dev["target"], dev["drafter"], None, dev["uniforms"],
                                    cfg.batch, cfg.positions)
    torch.cuda.synchronize()
    B.check_status_word(out)
    PU.compare_sampling(inp, out, range(cfg.rows), "linear", kept_ids=kid.cpu().numpy()).assert_ok()


def test_row_kernel_flag_and_route_query():
    """The same problem through the streaming kernel and, with RDK_FLAG_ROW_KERNEL, through the
    one-CTA-per-row kernel; rdk_sample_route names the kernel either call takes and why."""
    rdk = _rdk()
    B = rdk.binding
    cfg = W.tiny_config(N=20000, n=3000, rows=6, dtype="bf16", trials=4, rho=0.6, seed=91)
    inp = W.make_inputs(cfg)
    kid = inp["kept_ids"].cuda()
    idx = rdk.rdk_prepare_ids(kid, cfg.N)
    dev = {k: inp[k].cuda() for k in ("target", "drafter", "uniforms")}
    a = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_LINEAR, dev["target"], dev["drafter"], None, dev["uniforms"], cfg.batch, cfg.positions)
    b = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_LINEAR, dev["target"], dev["drafter"], None, dev["uniforms"], cfg.batch, cfg.positions,
                                  flags=B.RDK_FLAG_ROW_KERNEL)
    torch.cuda.synchronize()
    for o in (a, b):
        B.check_status_word(o)
        PU.compare_sampling(inp, o, range(cfg.rows), "linear").assert_ok()
    ws = a["_ws"]
    assert rdk.rdk_sample_route(idx, B.RDK_MODE_LINEAR, dev["target"], dev["drafter"], cfg.batch, cfg.positions, cfg.trials, ws)[0] == B.RDK_ROUTE_STREAM_KERNEL
    r, why = rdk.rdk_sample_route(idx, B.RDK_MODE_LINEAR, dev["target"], dev["drafter"], cfg.batch, cfg.positions, cfg.trials, ws,
                                  flags=B.RDK_FLAG_ROW_KERNEL)
    assert r == B.RDK_ROUTE_ROW_KERNEL and "FLAG" in why
    flat = torch.empty(cfg.rows * cfg.N + 8, dtype=torch.bfloat16, device="cuda")
    odd = flat[1: 1 + cfg.rows * cfg.N].view(cfg.rows, cfg.N)      # rows that do not start on 16-byte boundaries
    r, why = rdk.rdk_sample_route(idx, B.RDK_MODE_LINEAR, odd, dev["drafter"], cfg.batch, cfg.positions, cfg.trials, ws)
    assert r == B.RDK_ROUTE_ROW_KERNEL and "aligned" in why
    g = torch.Generator().manual_seed(1)
    shuffled = rdk.rdk_prepare_ids(kid[torch.randperm(cfg.n, generator=g).cuda()], cfg.N)
    r, why = rdk.rdk_sample_route(shuffled, B.RDK_MODE_LINEAR, dev["target"], dev["drafter"], cfg.batch, cfg.positions, cfg.trials, ws)
    assert r == B.RDK_ROUTE_ROW_KERNEL and "ascending" in why


def test_strided_rows_through_the_streaming_kernels():
    """Rows embedded in wider buffers (target stride a multiple of 8 elements, drafter stride even but
    not a multiple of 8, so the drafter rows start at varying 16-byte phases)."""
    rdk = _rdk()
    B = rdk.binding
    cfg = W.tiny_config(N=24576, n=5001, rows=40, dtype="bf16", trials=2, kept_rule="zipf", zipf_bias=True,
                        rho=0.7, seed=57)
    inp = W.make_inputs(cfg)
    tw = torch.zeros(cfg.rows, cfg.N + 24, dtype=torch.bfloat16)
    tw[:, : cfg.N] = inp["target"]
    dw = torch.zeros(cfg.rows, cfg.n + 5, dtype=torch.bfloat16)
    dw[:, : cfg.n] = inp["drafter"]
    idx = rdk.rdk_prepare_ids(inp["kept_ids"].cuda(), cfg.N)
    out = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_LINEAR, tw.cuda()[:, : cfg.N], dw.cuda()[:, : cfg.n], None,
                                    inp["uniforms"].cuda(), cfg.batch, cfg.positions)
    torch.cuda.synchronize()
    B.check_status_word(out)
    PU.compare_sampling(inp, out, range(cfg.rows), "linear").assert_ok()


@pytest.mark.parametrize("name,nrows", [("C2", 320), ("C3", 128), ("C4", 128)])
def test_full_size_configs_sampled_rows(name, nrows):
    """Full-size workloads in the launch configuration the benchmark times.  The checker recomputes every
    row of C2 and a seeded sample of 128 rows of C3 and C4 one by one (all per-row outputs of those rows
    are compared)."""
    cfg = W.CONFIGS[name]
    inp = W.make_inputs(cfg, device="cuda")
    rng = np.random.default_rng(cfg.seed)
    rows = (list(range(cfg.rows)) if nrows >= cfg.rows else
            sorted(set([0, cfg.rows - 1] + rng.choice(cfg.rows, nrows, replace=False).tolist())))
    rdk = _rdk()
    B = rdk.binding
    idx0 = rdk.rdk_prepare_ids(inp["kept_ids"], cfg.N)
    ws0 = B.sample_workspace(B.make_problem(idx0, inp["target"], inp["drafter"], cfg.batch, cfg.positions), B.RDK_MODE_LINEAR,
                             cfg.trials, "cuda")
    route, why = rdk.rdk_sample_route(idx0, B.RDK_MODE_LINEAR, inp["target"], inp["drafter"], cfg.batch, cfg.positions,
                                      cfg.trials, ws0)
    assert route == rdk.binding.RDK_ROUTE_STREAM_KERNEL, why
    t = _run_linear(cfg, inp, rows=rows, check_qtilde=False)
    t.assert_ok_at_scale(cfg.n)
    # properties that hold for every row at any size
    idx = rdk.rdk_prepare_ids(inp["kept_ids"], cfg.N)
    out = rdk.rdk_sample_and_verify(idx, rdk.binding.RDK_MODE_LINEAR, inp["target"], inp["drafter"], None,
                                    inp["uniforms"], cfg.batch, cfg.positions)
    torch.cuda.synchronize()
    a, R, S = out["alpha"].double(), out["residual_mass"].double(), out["S"].double()
    assert torch.all((a + R - 1).abs() < 2e-5)                      # Lemma 2.3: alpha = 1 - ||k||_1
    assert torch.all((S - 1).abs() < 1e-3) and torch.all(a > 0) and torch.all(a <= 1 + 1e-6)
    d = out["draft_token"].long()
    assert torch.all((d >= 0) & (d < cfg.N))
    ot = out["out_token"].long()
    acc = out["accepted"].bool()
    assert torch.all(ot[acc] == d[acc])
    assert torch.all((out["accept_prob"] >= 0) & (out["accept_prob"] <= 1))
    # acceptance frequency is consistent with the closed-form rate (binomial, 5 sigma)
    mean_alpha = a.mean().item()
    sigma = (a * (1 - a)).sum().sqrt().item() / cfg.rows
    assert abs(acc.double().mean().item() - mean_alpha) < 5 * sigma + 1e-3


def _masked_drafter(inp, cfg):
    """Scheme (a) of Sec. 5.2: the unpruned drafter's soft-max, zero outside the kept ids, not renormalised."""
    q_full = torch.softmax(inp["drafter_full"].float(), dim=-1)
    w = torch.zeros(cfg.rows, cfg.N, dtype=torch.float32, device=q_full.device)
    kid = inp["kept_ids"].long()
    w[:, kid] = q_full[:, kid]
    return w


def _check_w_as_given(rdk, cfg, inp, w, out, rows):
    """RDK_FLAG_W_AS_GIVEN against the checker's primitives with q~ = w, un-normalised: alpha (Definition 2.1), the
    draw in proportion to w, the rejection test and the residual (Algorithm 4 steps 4-8)."""
    t = PU.Tally()
    for r in rows:
        p = O.softmax(W.to_f64(inp["target"][r]))
        wr = W.to_f64(w[r])
        u = inp["uniforms"][r].cpu().numpy().astype(np.float64)
        assert abs(float(out["alpha"][r]) - O.acceptance_rate(p, wr)) < PU.ABS_TOL
        R, _ = O.residual(p, wr)
        assert abs(float(out["residual_mass"][r]) - R) < PU.ABS_TOL
        assert abs(float(out["S"][r]) - wr.sum()) < PU.ABS_TOL
        for k in range(cfg.trials):
            d = O.inverse_cdf(wr, u[k, 0])
            got_d = int(out["draft_token"][r * cfg.trials + k])
            if got_d != d:
                cdf = np.cumsum(wr)
                thr = u[k, 0] * cdf[-1]
                lo = cdf[got_d - 1] if got_d > 0 else 0.0
                assert min(abs(thr - lo), abs(thr - cdf[got_d])) <= PU.ABS_TOL * cdf[-1], (r, k, d, got_d)
                t.ambiguous_draft += 1
                continue
            a, acc = O.accept_test(p, wr, d, u[k, 1])
            assert abs(float(out["accept_prob"][r * cfg.trials + k]) - a) < 1e-4
            if bool(out["accepted"][r * cfg.trials + k]) != acc:
                assert abs(u[k, 1] * wr[d] - p[d]) <= PU.ABS_TOL * max(p[d], wr[d])
                t.ambiguous_accept += 1
                continue
            want = d if acc else O.residual_sample(p, wr, u[k, 2])
            got = int(out["out_token"][r * cfg.trials + k])
            if got != want:
                cr = np.cumsum(np.maximum(0.0, p - wr))
                thr = u[k, 2] * cr[-1]
                lo = cr[got - 1] if got > 0 else 0.0
                assert min(abs(thr - lo), abs(thr - cr[got])) <= PU.ABS_TOL * cr[-1], (r, k, want, got)
                t.ambiguous_residual += 1
        t.draws += cfg.trials
    return t


def test_pruning_without_redistribution_keeps_w_as_given():
    """Scheme (a) of Sec. 5.2 on a small problem, several trials per row: with RDK_FLAG_W_AS_GIVEN the sampler
    verifies against the masked, un-normalised drafter distribution; the flag is refused in the linear mode."""
    rdk = _rdk()
    B = rdk.binding
    cfg = W.tiny_config(N=5003, n=311, rows=7, dtype="bf16", trials=8, rho=0.8, seed=77)
    inp = W.make_inputs(cfg, device="cuda", with_full_drafter=True)
    idx = rdk.rdk_prepare_ids(inp["kept_ids"], cfg.N)
    w = _masked_drafter(inp, cfg)
    assert torch.all(w.sum(-1) < 0.999)                 # mass was pruned away: this is not TLI
    out = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_PRECOMPUTED_W, inp["target"], None, w, inp["uniforms"],
                                    cfg.batch, cfg.positions, flags=B.RDK_FLAG_W_AS_GIVEN)
    torch.cuda.synchronize()
    t = _check_w_as_given(rdk, cfg, inp, w, out, range(cfg.rows))
    t.assert_ok()
    # without the flag the same w is renormalised (TLI of the masked drafter): a different alpha
    out_n = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_PRECOMPUTED_W, inp["target"], None, w, inp["uniforms"],
                                      cfg.batch, cfg.positions)
    torch.cuda.synchronize()
    assert torch.all(out_n["alpha"] > out["alpha"] + 1e-4)
    with pytest.raises(Exception, match="W_AS_GIVEN"):
        rdk.rdk_sample_and_verify(idx, B.RDK_MODE_LINEAR, inp["target"], inp["drafter"], None, inp["uniforms"],
                                  cfg.batch, cfg.positions, flags=B.RDK_FLAG_W_AS_GIVEN)


def test_extreme_pruning_heavy_tailed_logits_three_schemes():
    """200k vocabulary, 500 kept tokens, Student-t logits (the shape of the synthetic experiment of Sec. 5.2):
    parity of the linear path on every row, and the two baselines next to it through the precomputed-w mode:
    TLI (w = q' scattered to the full vocabulary) and pruning without redistribution (w = the unpruned
    drafter's q masked to the kept ids, RDK_FLAG_W_AS_GIVEN)."""
    rdk = _rdk()
    B = rdk.binding
    cfg = W.CONFIGS["T1"]
    inp = W.make_inputs(cfg, device="cuda", with_full_drafter=True)
    rows = list(range(cfg.rows))
    t = _run_linear(cfg, inp, rows=rows, check_qtilde=False)
    t.assert_ok_at_scale(cfg.n)
    t.record("T1 linear, all rows")
    idx = rdk.rdk_prepare_ids(inp["kept_ids"], cfg.N)
    out_rdk = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_LINEAR, inp["target"], inp["drafter"], None, inp["uniforms"],
                                        cfg.batch, cfg.positions)
    # TLI: q' placed at the kept ids, zero elsewhere (generator-side scatter of the drafter soft-max)
    qp = torch.softmax(inp["drafter"].float(), dim=-1)
    w = torch.zeros(cfg.rows, cfg.N, dtype=torch.float32, device="cuda")
    w[:, inp["kept_ids"].long()] = qp
    out_tli = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_PRECOMPUTED_W, inp["target"], None, w, inp["uniforms"],
                                        cfg.batch, cfg.positions)
    wm = _masked_drafter(inp, cfg)
    out_prune = rdk.rdk_sample_and_verify(idx, B.RDK_MODE_PRECOMPUTED_W, inp["target"], None, wm, inp["uniforms"],
                                          cfg.batch, cfg.positions, flags=B.RDK_FLAG_W_AS_GIVEN)
    torch.cuda.synchronize()
    kappa = inp["kept_ids"].cpu().numpy()
    for r in rows[::8]:
        p = O.softmax(W.to_f64(inp["target"][r]))
        q_tli = O.tli_project(W.to_f64(w[r])[kappa], kappa, cfg.N)
        assert abs(float(out_tli["alpha"][r]) - O.acceptance_rate(p, q_tli)) < PU.ABS_TOL
    _check_w_as_given(rdk, cfg, inp, wm, out_prune, rows[::8])
    a_rdk, a_tli, a_prune = out_rdk["alpha"].double(), out_tli["alpha"].double(), out_prune["alpha"].double()
    # the first-order formula moves only about theta / N of the mass: both rates agree to ~1e-5 here
    assert torch.all((a_rdk - a_tli).abs() < 1e-4)
    # masking shrinks every kept probability, renormalising can only raise min(p, q) term by term
    assert torch.all(a_prune <= a_tli + 1e-6)


@pytest.mark.parametrize("dtype,N,n,kind", [("bf16", 5000, 900, "logits"), ("f32", 1001, 77, "logits"),
                                            ("bf16", 12808, 2000, "probs")])
def test_linear_with_a_separate_prior(dtype, N, n, kind):
    """Eq. rdk-taylor with a prior in place of p (per-row priors and one shared prior row), checked
    against the checker row by row: q~, theta, S element-wise, then draws, rejection test, alpha and
    residual against the true target."""
    rdk = _rdk()
    cfg = W.tiny_config(N=N, n=n, rows=5, dtype=dtype, trials=8, rho=0.7, seed=N + 3, drafter_kind=kind)
    inp = W.make_inputs(cfg)
    g = torch.Generator().manual_seed(N)
    noise = torch.randn(cfg.rows, cfg.N, generator=g) * 1.5
    per_row = (inp["target"].float() * 0.8 + noise).to(inp["target"].dtype)      # a blurred view of the target
    shared = per_row[0].clone().contiguous()
    idx = rdk.rdk_prepare_ids(inp["kept_ids"].cuda(), cfg.N)
    kappa = inp["kept_ids"].numpy()
    for prior in (per_row, shared):
        out = rdk.rdk_sample_and_verify_prior(idx, inp["target"].cuda(), prior.cuda(), inp["drafter"].cuda(),
                                              inp["uniforms"].cuda(), cfg.batch, cfg.positions, KIND[kind])
        qt, theta, S = rdk.rdk_redistribute_linear_prior(idx, inp["target"].cuda(), prior.cuda(), inp["drafter"].cuda(),
                                                         cfg.batch, cfg.positions, KIND[kind])
        torch.cuda.synchronize()
        rdk.binding.check_status_word(out)
        PU.compare_sampling(inp, out, range(cfg.rows), "linear", prior=prior).assert_ok()
        refs = {}
        for r in range(cfg.rows):
            pr = W.to_f64(prior if prior.dim() == 1 else prior[r])
            refs[r] = O.rdk_row(W.to_f64(inp["target"][r]), W.to_f64(inp["drafter"][r]), kappa, np.zeros((1, 4)), "linear",
                                drafter_kind=kind, prior=pr)
            assert PU.close(float(theta[r]), refs[r]["theta"], dtype == "bf16")
            assert PU.close(float(S[r]), refs[r]["S"], dtype == "bf16")
        PU.compare_qtilde(qt, refs, dtype == "bf16")
    # with the target itself as the prior the call reduces to the plain linear mode
    a = rdk.rdk_sample_and_verify_prior(idx, inp["target"].cuda(), inp["target"].cuda(), inp["drafter"].cuda(),
                                        inp["uniforms"].cuda(), cfg.batch, cfg.positions, KIND[kind])
    torch.cuda.synchronize()
    PU.compare_sampling(inp, a, range(cfg.rows), "linear").assert_ok()
