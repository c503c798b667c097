"""GPU-vs-oracle parity through the C ABI (see tests/parity.py for the comparison rules)."""

import numpy as np
import pytest

import fsd_inputs as gi
from oracle import fsd_oracle as orc
from tests import parity

pytestmark = pytest.mark.gpu


def _check(c, **kw):
    return parity.check_chain(c.target, c.draft, c.draft_tokens, c.u_accept, c.u_sample, c.dtype, **kw)


# --------------------------------------------------------------------------- #
# the five named workloads
# --------------------------------------------------------------------------- #
def test_config1_all_divergences_thresholds_and_compare_ops():
    c = gi.make_config("c1")
    for div in ("js", "kl", "tv"):
        for T in gi.CONFIGS["c1"].thresholds:
            for cmp in ("lt", "le"):
                r = _check(c, div=div, T=T, cmp=cmp)
                assert r["max_err"] <= 1e-5


def test_config2_fsd_and_sd_threshold_sweep():
    c = gi.make_config("c2")
    lens = []
    for T in gi.CONFIGS["c2"].thresholds:
        r = _check(c, mode="fsd", T=T)
        lens.append(r["accept_len"])
        assert r["max_err"] <= 1e-4
    assert all((b >= a).all() for a, b in zip(lens, lens[1:]))       # larger T never accepts less
    assert lens[0].max() == 0 and lens[-1].min() == c.gamma
    _check(c, mode="sd", T=0.0)
    for T in (0.0, 2.0 / 7):
        _check(c, mode="rfsd", T=T)
    for sample in ("greedy",):
        _check(c, mode="fsd", T=1.0 / 7, sample=sample)
        _check(c, mode="sd", sample=sample)


def test_config3_zipf_with_disjoint_drafts():
    c = gi.make_config("c3")
    for T in gi.CONFIGS["c3"].thresholds:
        r = _check(c, T=T)
        assert r["max_err"] <= 1e-4
    assert c.disjoint.any()
    r = _check(c, div="kl", T=0.3)
    r = _check(c, div="tv", T=0.3)
    # the strict and the relaxed ratio rule (Eq. 1-3, Eq. 6) at a full LLM vocabulary
    _check(c, mode="sd")
    _check(c, mode="rfsd", T=0.1)
    _check(c, mode="sd", sample="greedy")


def test_config4_headline_shape():
    c = gi.make_config("c4")
    r = _check(c, T=0.2)
    assert r["max_err"] <= 1e-4
    assert len(set(r["accept_len"].tolist())) > 2                    # the workload is not degenerate
    _check(c, T=0.2, cmp="le")
    _check(c, div="kl", T=0.2)
    _check(c, div="tv", T=0.2)
    _check(c, mode="sd")


@pytest.mark.parametrize("gamma", [10, 15, 20])
def test_paper_candidate_lengths_at_a_full_vocabulary(gamma):
    """The candidate lengths the paper runs (Appendix F: 5, 10, 15, 20) on the headline vocabulary;
    a small batch keeps the oracle affordable."""
    c = gi.make_chain(3, gamma, 152064, dtype="bf16", recipe="zipf", sigma=(0.2, 2.0), sigma_mode="uniform",
                      disjoint_frac=0.1, workload_id=400 + gamma)
    r = _check(c, T=0.2)
    assert r["max_err"] <= 1e-4
    _check(c, mode="sd")
    _check(c, mode="rfsd", T=0.2)


@pytest.mark.parametrize("dtype,V", [("bf16", 32776), ("f32", 16388), ("bf16", 65544), ("bf16", 131080)])
def test_slices_of_unequal_stage_counts_within_a_group(dtype, V):
    """Row lengths that split over a group of virtual CTAs into slices of which some need one ring
    stage more than the others, with more pairs than the groups take in their first rounds: the
    members of a group must still agree on which pair comes next."""
    c = gi.make_chain(16, 8, V, dtype=dtype, recipe="zipf", sigma=(0.2, 1.5), sigma_mode="uniform",
                      disjoint_frac=0.1, workload_id=420)
    r = _check(c, T=0.2)
    assert not (r["gpu"].row_status & 2).any()
    _check(c, div="tv", T=0.3)
    if V == 32776:
        t = gi.make_tree(4, 40, V, dtype=dtype, sigma=0.6, max_depth=5, workload_id=421)
        parity.check_tree(t, T=0.1)


def test_config5_tree():
    c = gi.make_config("c5")
    for T in gi.CONFIGS["c5"].thresholds:
        parity.check_tree(c, T=T)


# --------------------------------------------------------------------------- #
# small, odd and degenerate shapes
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [1, 2, 7, 8, 33, 1000, 4099, 20000])
def test_odd_vocabulary_sizes(dtype, V):
    c = gi.make_chain(3, 2, V, dtype=dtype, recipe="spike", sigma=(0.3, 1.0), workload_id=100 + V)
    for div in ("js", "kl", "tv"):
        _check(c, div=div, T=0.1)
    _check(c, mode="sd")
    _check(c, mode="rfsd", T=0.05)


def test_gamma_one_and_long_chains():
    for gamma in (1, 20, 70):
        c = gi.make_chain(2, gamma, 512, dtype="bf16", recipe="zipf", sigma=(0.2, 0.6), sigma_mode="uniform",
                          workload_id=200 + gamma)
        _check(c, T=0.05)
        _check(c, T=10.0)


def test_identical_rows_and_threshold_zero():
    c = gi.make_chain(4, 3, 4096, dtype="bf16", recipe="spike", sigma=(0.5,), workload_id=300)
    c.draft[0, 0] = c.target[0, 0]
    c.draft[0, 1] = c.target[0, 1]
    c.draft[2, 0] = c.target[2, 0]
    r = _check(c, T=0.0, cmp="le")
    assert r["accept_len"].tolist() == [2, 0, 1, 0]
    assert r["gpu"].divergence[0, 0] == 0.0 and r["gpu"].divergence[2, 0] == 0.0
    r = _check(c, T=0.0, cmp="lt")
    assert (r["accept_len"] == 0).all()
    for div in ("kl", "tv"):
        r = _check(c, T=0.0, cmp="le", div=div)
        assert r["gpu"].divergence[0, 1] == 0.0


def test_masked_logits_and_disjoint_supports():
    c = gi.make_chain(3, 2, 1024, dtype="f32", recipe="spike", sigma=(0.5,), workload_id=301)
    c.target[0, 0, 512:] = -np.inf
    c.draft[0, 0, :512] = -np.inf                 # disjoint: JS = ln 2, TV = 1, KL = inf
    c.target[1, 1, ::3] = -np.inf                 # masked target entries only
    c.draft[2, 0, 5::7] = -np.inf                 # masked draft entries: KL = inf
    for div in ("js", "kl", "tv"):
        r = _check(c, div=div, T=0.7)
    r = _check(c, div="js", T=0.7)
    assert abs(r["gpu"].divergence[0, 0] - np.log(2.0)) < 1e-6
    r = _check(c, div="kl", T=100.0)
    assert np.isposinf(r["gpu"].divergence[0, 0]) and np.isposinf(r["gpu"].divergence[2, 0])
    _check(c, mode="sd")


def test_nonfinite_rows_are_flagged_not_propagated():
    c = gi.make_chain(4, 3, 2048, dtype="f32", recipe="spike", sigma=(0.5,), workload_id=302)
    c.draft[0, 1, 17] = np.nan
    c.target[1, 0, 3] = np.inf
    c.target[2, 3, :] = -np.inf                   # the bonus row of row 2 has no finite entry
    r = _check(c, T=100.0)
    assert r["gpu"].row_status.tolist() == [1, 1, 1, 0]
    assert r["accept_len"].tolist() == [1, 0, 3, 3]
    assert r["gpu"].next_token[1] == -1 and r["gpu"].next_token[2] == -1
    _check(c, mode="sd")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_wide_dynamic_range_moves_the_reference(dtype):
    """Rows whose largest logits come late and far above the first ones (masked prefixes, late
    spikes, steep ramps): whatever reference a streaming softmax starts from has to move."""
    B, gamma, V = 4, 3, 40000
    c = gi.make_chain(B, gamma, V, dtype=dtype, recipe="spike", sigma=(0.5, 1.0), workload_id=306)
    f32 = dtype == "f32"
    t = c.target if f32 else gi.bf16_bits_to_f32(c.target)
    d = c.draft if f32 else gi.bf16_bits_to_f32(c.draft)
    k = np.arange(V, dtype=np.float32)
    t[0, :, :9000] = -np.inf                      # nothing finite for the first stages
    d[0, :, :13000] = -np.inf
    t[1, :, 30011:30014] += 90.0                  # late spikes: 130 binades above the rest
    d[1, :, 39990:] += 75.0
    t[2] += (k * 0.01 - 200.0)                    # +-200 nats ramp: the reference moves again and again
    d[2] += (k * 0.0125 - 250.0)
    t[3] -= k * 0.01                              # falling ramp: the first reference stays
    d[3, :, 1::2] = -np.inf
    d[3, :, -1] = 300.0                           # and one jump of > 126 binades at the very end
    if not f32:
        c.target[:] = gi.f32_to_bf16_bits(t)
        c.draft[:] = gi.f32_to_bf16_bits(d)
    for div in ("js", "kl", "tv"):
        _check(c, div=div, T=0.3)
    _check(c, mode="rfsd", T=0.3)


def test_uniform_extremes_for_sampling():
    c = gi.make_chain(6, 2, 5000, dtype="bf16", recipe="zipf", sigma=(0.5,), workload_id=303)
    c.u_sample[:] = np.array([0.0, np.nextafter(np.float32(1), np.float32(0)), 0.5, 1e-7, 0.999, 0.25], np.float32)
    _check(c, T=0.0)
    _check(c, T=10.0)
    c.u_accept[:] = 0.0
    _check(c, mode="sd")


def test_fsd_outputs_do_not_depend_on_tokens_or_accept_uniforms():
    c = gi.make_chain(4, 4, 3000, dtype="bf16", recipe="spike", sigma=(0.2, 1.5), sigma_mode="uniform", workload_id=304)
    a = parity.run_chain_gpu(c.target, c.draft, c.draft_tokens, c.u_accept, c.u_sample, c.dtype, T=0.1)
    b = parity.run_chain_gpu(c.target, c.draft, None, None, c.u_sample, c.dtype, T=0.1)
    assert np.array_equal(a.accept_len, b.accept_len) and np.array_equal(a.next_token, b.next_token)
    assert np.array_equal(a.divergence, b.divergence)
    # bit-reproducible from run to run
    a2 = parity.run_chain_gpu(c.target, c.draft, c.draft_tokens, c.u_accept, c.u_sample, c.dtype, T=0.1)
    assert np.array_equal(a.divergence, a2.divergence) and np.array_equal(a.next_token, a2.next_token)


@pytest.mark.parametrize("dtype,V", [("f32", 100000), ("f32", 152064), ("bf16", 200008), ("bf16", 256000)])
def test_vocabularies_that_need_groups_of_more_than_eight(dtype, V):
    """Rows too long for eight virtual CTAs' on-chip capacity (fp32 above 81920 entries, bf16 above
    163840) are streamed by larger groups (up to sixteen)."""
    c = gi.make_chain(5, 4, V, dtype=dtype, recipe="zipf", sigma=(0.3, 1.5), sigma_mode="uniform",
                      disjoint_frac=0.1, workload_id=309)
    for div in ("js", "kl", "tv"):
        _check(c, div=div, T=0.25)
    _check(c, mode="rfsd", T=0.25)


@pytest.mark.parametrize("V,sizes", [(4096, (1, 2, 3, 5, 16)), (32000, (2, 3, 7, 11, 16)), (152064, (8, 9, 13, 16))])
def test_every_group_size_gives_the_same_answers(V, sizes):
    """The streaming kernel splits a pair over a group of thread blocks whose size the library
    chooses; forced to other sizes (slices of one to five ring stages, even and uneven splits,
    more and fewer groups than pairs) the kernel must agree with the oracle all the same, and
    decisions and tokens must not depend on the size."""
    from paper_2502_20704_b200 import binding as fsd

    c = gi.make_chain(6, 5, V, dtype="bf16", recipe="zipf", sigma=(0.2, 1.5), sigma_mode="uniform",
                      disjoint_frac=0.1, workload_id=430)
    base = _check(c, T=0.2)["gpu"]
    try:
        for size in sizes:
            assert fsd.fsd_set_group_size(size) == 0
            for div in ("js", "kl", "tv"):
                _check(c, div=div, T=0.2)
            r = _check(c, T=0.2)["gpu"]
            assert np.allclose(r.divergence, base.divergence, rtol=0, atol=2e-6)
            clear = (np.abs(base.divergence - 0.2) > 1e-5).all(axis=1)      # rows with no divergence at the threshold
            assert np.array_equal(r.accept_len[clear], base.accept_len[clear])
            assert np.array_equal(r.next_token[clear], base.next_token[clear])
    finally:
        fsd.fsd_set_group_size(0)
    assert fsd.fsd_set_group_size(17) != 0 and fsd.fsd_set_group_size(-1) != 0


def test_calls_on_two_streams_with_their_own_workspaces_do_not_disturb_each_other():
    """Two workloads verified at once on two streams (separate workspaces, as the header asks):
    each must give exactly what it gives alone; a workspace reused call after call must, too."""
    import torch
    from paper_2502_20704_b200 import binding as fsd

    ca = gi.make_chain(24, 6, 36000, dtype="bf16", recipe="zipf", sigma=(0.4, 1.2), sigma_mode="uniform", workload_id=307)
    cb = gi.make_chain(16, 9, 52000, dtype="bf16", recipe="spike", sigma=(0.2, 2.0), sigma_mode="uniform", workload_id=308)
    alone = [parity.run_chain_gpu(c.target, c.draft, None, None, c.u_sample, c.dtype, T=0.15) for c in (ca, cb)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    jobs = []
    for c in (ca, cb):
        B, g1, V = c.target.shape
        gamma = g1 - 1
        opts = fsd.make_opts(dtype=c.dtype, T=0.15)
        wsb = fsd.fsd_workspace_bytes(B, gamma, V, opts)
        jobs.append(dict(B=B, gamma=gamma, V=V, opts=opts, wsb=wsb,
                         t=parity.to_device(c.target, c.dtype), d=parity.to_device(c.draft, c.dtype),
                         us=parity.to_device(c.u_sample, c.dtype),
                         acc=torch.empty(B, dtype=torch.int32, device="cuda"),
                         tok=torch.empty(B, dtype=torch.int32, device="cuda"),
                         D=torch.empty(B, gamma, dtype=torch.float32, device="cuda"),
                         st=torch.empty(B, dtype=torch.int32, device="cuda"),
                         ws=torch.full((wsb,), 0xCD, dtype=torch.uint8, device="cuda")))
    torch.cuda.synchronize()
    for rep in range(6):                              # interleaved: both streams always have work queued
        for j, s in zip(jobs, streams):
            rc = fsd.fsd_verify_chain(j["t"], j["d"], None, None, j["us"], j["B"], j["gamma"], j["V"], j["opts"],
                                      j["acc"], j["tok"], j["D"], j["st"], j["ws"], j["wsb"], s.cuda_stream)
            assert rc == 0, fsd.fsd_status_string(rc)
    torch.cuda.synchronize()
    for j, ref in zip(jobs, alone):
        assert np.array_equal(j["acc"].cpu().numpy(), ref.accept_len)
        assert np.array_equal(j["tok"].cpu().numpy(), ref.next_token)
        assert np.array_equal(j["D"].cpu().numpy(), ref.divergence)
        assert not j["st"].cpu().numpy().any()


def test_out_of_range_draft_token_is_rejected_in_sd_mode():
    c = gi.make_chain(2, 3, 512, dtype="f32", recipe="spike", sigma=(0.1,), workload_id=305)
    c.draft_tokens[0, 1] = 512
    c.draft_tokens[1, 0] = -1
    c.u_accept[:] = 0.0
    r = _check(c, mode="sd")
    assert r["accept_len"].tolist() == [1, 0]


# --------------------------------------------------------------------------- #
# trees
# --------------------------------------------------------------------------- #
def test_chain_shaped_tree_matches_chain_call():
    B, N, V = 3, 5, 4096
    parent = np.tile(np.arange(-1, N - 1, dtype=np.int32), (B, 1))
    t = gi.make_tree(B, N, V, dtype="bf16", sigma=0.6, workload_id=400, parent=parent)
    for T in (0.02, 0.045, 0.3):
        g = parity.run_tree_gpu(t.target, t.draft, t.parent, t.u_sample, N, t.dtype, T=T)
        c = parity.run_chain_gpu(t.target, t.draft, None, None, t.u_sample, t.dtype, T=T)
        assert np.array_equal(g.accept_len, c.accept_len) and np.array_equal(g.next_token, c.next_token)
        assert np.array_equal(g.divergence, c.divergence)


def test_largest_trees_chain_shaped_and_bushy():
    """The allowed maximum of 1024 nodes: a chain-shaped tree (depth 1024, the worst case for the
    path selection) and a bushy random one, against the oracle."""
    N, V = 1024, 1024
    chain_parent = np.arange(-1, N - 1, dtype=np.int32)[None, :]
    t = gi.make_tree(2, N, V, dtype="f32", sigma=0.05, max_depth=N, workload_id=402, parent=chain_parent)
    for T in (1e-3, 2e-3, 1.0):
        g, o = parity.check_tree(t, T=T)
    assert g.accept_len.max() == N                       # with T = 1 the whole chain passes
    t = gi.make_tree(2, N, V, dtype="f32", sigma=0.3, max_depth=9, max_children=4, workload_id=403)
    for T in (0.02, 0.05, 1.0):
        parity.check_tree(t, T=T)


def test_tree_max_depth_and_bad_parent():
    t = gi.make_tree(3, 12, 2048, dtype="f32", sigma=0.3, max_depth=5, workload_id=401)
    t.parent[1, 4] = 4                           # a node naming itself as parent
    for depth in (1, 2, 5):
        g = parity.run_tree_gpu(t.target, t.draft, t.parent, t.u_sample, depth, t.dtype, T=5.0)
        o = orc.verify_tree(t.target, t.draft, t.parent, t.u_sample, depth, dtype=t.dtype, T=5.0,
                            band=parity.SAMPLE_BAND)
        assert np.array_equal(g.accept_len, o.accept_len) and np.array_equal(g.path, o.path)
        assert np.array_equal(g.next_token, o.next_token) and np.array_equal(g.row_status, o.row_status)
        assert g.row_status[1] & 4 and g.accept_len[1] == 0 and g.next_token[1] == -1
        assert g.accept_len.max() <= depth
        parity.compare_divergence(g.divergence, o.divergence, 1e-5)


def test_a_verify_call_can_be_captured_in_a_cuda_graph_and_replayed():
    """A decoding loop captures its steps once and replays them: the call (a memset, the cooperative
    streaming kernel, the finish kernel) must be capturable after one ordinary call, and a replay on
    new inputs in the same buffers must give what an ordinary call gives."""
    import torch
    from paper_2502_20704_b200 import binding as fsd

    cs = [gi.make_chain(8, 5, 50000, dtype="bf16", recipe="zipf", sigma=(0.3, 1.5), sigma_mode="uniform", workload_id=450 + k)
          for k in range(2)]
    want = [parity.check_chain(c.target, c.draft, c.draft_tokens, c.u_accept, c.u_sample, c.dtype, T=0.15)["gpu"] for c in cs]
    B, g1, V = cs[0].target.shape
    gamma = g1 - 1
    opts = fsd.make_opts(dtype="bf16", T=0.15)
    t = parity.to_device(cs[0].target, "bf16")
    d = parity.to_device(cs[0].draft, "bf16")
    us = parity.to_device(cs[0].u_sample, "bf16")
    acc = torch.zeros(B, dtype=torch.int32, device="cuda")
    tok = torch.zeros(B, dtype=torch.int32, device="cuda")
    st = torch.zeros(B, dtype=torch.int32, device="cuda")
    D = torch.zeros(B, gamma, dtype=torch.float32, device="cuda")
    wsb = fsd.fsd_workspace_bytes(B, gamma, V, opts)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        assert fsd.fsd_verify_chain(t, d, None, None, us, B, gamma, V, opts, acc, tok, D, st, ws, wsb, side.cuda_stream) == 0
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        rc = fsd.fsd_verify_chain(t, d, None, None, us, B, gamma, V, opts, acc, tok, D, st, ws, wsb, side.cuda_stream)
    assert rc == 0
    for k in (1, 0, 1):
        t.copy_(parity.to_device(cs[k].target, "bf16"))
        d.copy_(parity.to_device(cs[k].draft, "bf16"))
        us.copy_(parity.to_device(cs[k].u_sample, "bf16"))
        acc.fill_(-7); tok.fill_(-7); D.fill_(-7.0)
        graph.replay()
        torch.cuda.synchronize()
        assert np.array_equal(acc.cpu().numpy(), want[k].accept_len)
        assert np.array_equal(tok.cpu().numpy(), want[k].next_token)
        assert np.array_equal(D.cpu().numpy().view(np.uint32), want[k].divergence.view(np.uint32))


def test_calls_of_changing_shapes_queued_on_one_workspace():
    """Calls of different shapes (so different group sizes, grids and record counts) queued back to
    back on one stream and one workspace, without a synchronisation in between: nothing one call
    leaves in the workspace (messages, counters, records) may reach the next.  Each call must give
    exactly what it gives alone on a fresh workspace."""
    import torch
    from paper_2502_20704_b200 import binding as fsd

    shapes = [(3, 4, 32000), (16, 5, 4096), (2, 8, 152064), (40, 3, 8192), (1, 1, 50000), (7, 6, 65544)]
    cases = [gi.make_chain(B, g, V, dtype="bf16", recipe="zipf", sigma=(0.3, 1.5), sigma_mode="uniform",
                           disjoint_frac=0.1, workload_id=460 + k) for k, (B, g, V) in enumerate(shapes)]
    alone = [parity.run_chain_gpu(c.target, c.draft, None, None, c.u_sample, c.dtype, T=0.15) for c in cases]
    opts = fsd.make_opts(dtype="bf16", T=0.15)
    wsb = max(fsd.fsd_workspace_bytes(B, g, V, opts) for B, g, V in shapes)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    ws.fill_(0xAB)
    stream = torch.cuda.current_stream().cuda_stream
    dev, outs = [], []
    for c in cases:
        B, g1, V = c.target.shape
        dev.append((parity.to_device(c.target, "bf16"), parity.to_device(c.draft, "bf16"), parity.to_device(c.u_sample, "bf16")))
        outs.append((torch.full((B,), -7, dtype=torch.int32, device="cuda"), torch.full((B,), -7, dtype=torch.int32, device="cuda"),
                     torch.full((B, g1 - 1), -7.0, dtype=torch.float32, device="cuda"), torch.full((B,), -7, dtype=torch.int32, device="cuda")))
    torch.cuda.synchronize()
    order = [0, 1, 2, 3, 4, 5, 5, 2, 0, 4, 3, 1, 2, 2, 4]
    for k in order:
        B, g1, V = cases[k].target.shape
        t, d, us = dev[k]
        acc, tok, D, st = outs[k]
        assert fsd.fsd_verify_chain(t, d, None, None, us, B, g1 - 1, V, opts, acc, tok, D, st, ws, wsb, stream) == 0
    torch.cuda.synchronize()
    for k, a in enumerate(alone):
        acc, tok, D, st = outs[k]
        assert np.array_equal(acc.cpu().numpy(), a.accept_len) and np.array_equal(tok.cpu().numpy(), a.next_token)
        assert np.array_equal(st.cpu().numpy(), a.row_status)
        assert np.array_equal(D.cpu().numpy().view(np.uint32), a.divergence.view(np.uint32))


def test_residual_draw_when_the_two_rows_agree_almost_everywhere():
    """SD rule, a rejection between two rows that are identical except for a handful of entries.
    Every identical entry then has exactly the same weight in both rows and carries residual mass
    only through the tiny difference of the two normalisers: whether it counts hangs on the exact
    ratio of the normalisers, which the one-pass form of the residual sums cannot decide from its
    estimate, so these rows must go through the second pass -- and agree with the oracle there."""
    rng = np.random.default_rng(471)
    B, gamma, V = 6, 3, 4096
    base = (-1.1 * np.log(np.arange(1, V + 1)) + 0.3 * rng.standard_normal((B, gamma + 1, V))).astype(np.float32)
    target = gi.bf16_bits_to_f32(gi.f32_to_bf16_bits(base))
    draft = target[:, :gamma, :].copy()
    tokens = np.zeros((B, gamma), dtype=np.int32)
    u_acc = np.full((B, gamma), 0.5, dtype=np.float32)
    for b in range(B):
        j1, j2 = 1000 + 17 * b, 2000 + 29 * b          # low-probability entries
        draft[b, 0, j1] += 0.5 * (b + 1)                # q > p there: proposing j1 is rejected for u close to 1
        draft[b, 0, j2] -= 0.25
        tokens[b, 0] = j1
        u_acc[b, 0] = 0.999
    tbits, dbits = gi.f32_to_bf16_bits(target), gi.f32_to_bf16_bits(draft)
    u_sample = rng.random(B).astype(np.float32)
    r = parity.check_chain(tbits, dbits, tokens, u_acc, u_sample, "bf16", mode="sd", T=0.2)
    assert (r["gpu"].accept_len == 0).all()
    parity.check_chain(tbits, dbits, tokens, u_acc, u_sample, "bf16", mode="rfsd", T=0.0)

