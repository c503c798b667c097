"""Pins for the CPU oracle: each test fixes the oracle to something other than itself --
hand-derived values, closed forms, invariants, brute force on tiny vocabularies."""

import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import fsd_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
LN2 = math.log(2.0)


def _logits_of(p):
    """float32 logits whose softmax is p (zero probability -> -inf)."""
    with np.errstate(divide="ignore"):
        return np.log(np.asarray(p, dtype=np.float64)).astype(np.float32)


def _load_golden():
    rows = []
    with open(os.path.join(GOLDEN, "divergence_small.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, p, q, kl, js, tv = [s.strip() for s in line.split(";")]
            pv = [float(Fraction(x)) for x in p.split()]
            qv = [float(Fraction(x)) for x in q.split()]
            rows.append((name, pv, qv, float(kl), float(js), float(tv)))
    return rows


# --------------------------------------------------------------------------- #
# divergences: hand-derived values (Appendix C definitions)
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("row", _load_golden(), ids=lambda r: r[0])
def test_divergence_golden_probs(row):
    _, p, q, kl, js, tv = row
    assert orc.divergence_probs(p, q, "kl") == pytest.approx(kl, abs=1e-14)
    assert orc.divergence_probs(p, q, "js") == pytest.approx(js, abs=1e-14)
    assert orc.divergence_probs(p, q, "tv") == pytest.approx(tv, abs=1e-14)


@pytest.mark.parametrize("row", _load_golden(), ids=lambda r: r[0])
def test_divergence_golden_through_softmax(row):
    """Same values reached from logits = ln p (+ a constant), through the softmax step."""
    _, p, q, kl, js, tv = row
    a = _logits_of(p) + np.float32(3.0)
    b = _logits_of(q) - np.float32(1.5)
    # float32 storage of ln p perturbs p by ~1e-7 relative
    assert orc.divergence_logits(a, b, "kl") == pytest.approx(kl, abs=5e-7)
    assert orc.divergence_logits(a, b, "js") == pytest.approx(js, abs=5e-7)
    assert orc.divergence_logits(a, b, "tv") == pytest.approx(tv, abs=5e-7)


def test_kl_direction_is_target_given_draft():
    # KL(p||q) != KL(q||p) for case A; the chain call must use target as the first operand
    p, q = [0.5, 0.5], [0.25, 0.75]
    target = np.stack([_logits_of(p), _logits_of(p)])[None]          # [1, 2, V]
    draft = _logits_of(q)[None, None]                                # [1, 1, V]
    r = orc.verify_chain(target, draft, None, None, np.zeros(1, np.float32), dtype="f32", div="kl", T=1.0)
    assert r.divergence[0, 0] == pytest.approx(0.14384103622589046, abs=5e-7)
    assert abs(r.divergence[0, 0] - 0.13081203594113696) > 1e-3


# --------------------------------------------------------------------------- #
# closed forms, bounds and invariants
# --------------------------------------------------------------------------- #
def _rand_probs(rng, V, zeros=0):
    p = rng.gamma(0.3, size=V) + 1e-300
    if zeros:
        p[rng.choice(V, zeros, replace=False)] = 0.0
    return p / p.sum()


def test_identical_distributions_have_zero_divergence():
    rng = np.random.default_rng(1)
    for V in (2, 5, 33, 1000):
        a = rng.normal(size=V).astype(np.float32) * 4
        for kind in ("js", "kl", "tv"):
            assert orc.divergence_logits(a, a.copy(), kind) == 0.0


def test_disjoint_supports_reach_the_upper_bounds():
    rng = np.random.default_rng(2)
    V = 64
    a = rng.normal(size=V).astype(np.float32)
    b = rng.normal(size=V).astype(np.float32)
    a[V // 2:] = -np.inf
    b[:V // 2] = -np.inf
    assert orc.divergence_logits(a, b, "js") == pytest.approx(LN2, abs=1e-15)
    assert orc.divergence_logits(a, b, "tv") == pytest.approx(1.0, abs=1e-15)
    assert orc.divergence_logits(a, b, "kl") == math.inf


def test_bounds_symmetry_and_textbook_inequalities():
    rng = np.random.default_rng(3)
    for trial in range(200):
        V = int(rng.integers(2, 40))
        p = _rand_probs(rng, V, zeros=int(rng.integers(0, V // 2)))
        q = _rand_probs(rng, V)
        js, tv, kl = (orc.divergence_probs(p, q, k) for k in ("js", "tv", "kl"))
        assert 0.0 <= js <= LN2 + 1e-15
        assert 0.0 <= tv <= 1.0 + 1e-15
        assert kl >= 0.0
        assert js == pytest.approx(orc.divergence_probs(q, p, "js"), abs=1e-15)
        assert tv == pytest.approx(orc.divergence_probs(q, p, "tv"), abs=1e-15)
        assert tv <= math.sqrt(kl / 2.0) + 1e-12            # Pinsker
        assert js <= LN2 * tv + 1e-12                        # JS <= ln2 * TV
        assert js >= tv * tv / 2.0 - 1e-12                   # Pinsker applied to both halves of JS


def test_js_equals_entropy_form():
    """JS = H(m) - (H(p) + H(q))/2, an identity the term-by-term definition must satisfy."""
    rng = np.random.default_rng(4)
    H = lambda x: -sum(v * math.log(v) for v in x if v > 0)
    for _ in range(50):
        V = int(rng.integers(2, 50))
        p, q = _rand_probs(rng, V), _rand_probs(rng, V, zeros=1)
        m = 0.5 * (p + q)
        assert orc.divergence_probs(p, q, "js") == pytest.approx(H(m) - 0.5 * H(p) - 0.5 * H(q), abs=1e-13)


def test_shift_and_permutation_invariance():
    rng = np.random.default_rng(5)
    V = 257
    a = (rng.normal(size=V) * 3).astype(np.float32)
    b = (a + rng.normal(size=V)).astype(np.float32)
    perm = rng.permutation(V)
    for kind in ("js", "kl", "tv"):
        d = orc.divergence_logits(a, b, kind)
        # a power-of-two shift keeps the float32 logits exact
        assert orc.divergence_logits(a + np.float32(16.0), b - np.float32(8.0), kind) == pytest.approx(d, abs=1e-6)
        assert orc.divergence_logits(a[perm].copy(), b[perm].copy(), kind) == pytest.approx(d, abs=1e-13)


def test_softmax_properties():
    rng = np.random.default_rng(6)
    a = rng.normal(size=500).astype(np.float32)
    p, st = orc.softmax(a)
    assert st == 0
    assert abs(p.sum() - 1.0) < 1e-15
    naive = np.exp(a.astype(np.float64))
    naive /= naive.sum()
    assert np.allclose(p, naive, rtol=1e-13, atol=0)
    p2, _ = orc.softmax(a + np.float32(64.0))                # exact shift for these magnitudes? not always:
    a64 = (a.astype(np.float64) + 64.0).astype(np.float32)   # compare against the shifted values actually stored
    n2 = np.exp(a64.astype(np.float64) - a64.max())
    assert np.allclose(p2, n2 / n2.sum(), rtol=1e-13, atol=0)
    # large magnitudes do not overflow
    big = np.array([1000.0, 999.0, -1000.0], dtype=np.float32)
    pb, st = orc.softmax(big)
    assert st == 0 and pb[0] == pytest.approx(1 / (1 + math.exp(-1)), rel=1e-14) and pb[2] == 0.0


def test_softmax_bf16_widening_is_exact():
    bits = np.array([0x3F80, 0x4000, 0xBF80, 0x0000], dtype=np.uint16)    # 1, 2, -1, 0
    p, st = orc.softmax(bits, "bf16")
    e = np.exp(np.array([1.0, 2.0, -1.0, 0.0]))
    assert st == 0 and np.allclose(p, e / e.sum(), rtol=1e-14)


def test_nonfinite_rows_are_flagged():
    for bad in (np.nan, np.inf):
        a = np.array([0.0, bad, 1.0], dtype=np.float32)
        p, st = orc.softmax(a)
        assert st == orc.ST_NONFINITE and np.isnan(p).all()
    p, st = orc.softmax(np.full(4, -np.inf, dtype=np.float32))
    assert st == orc.ST_NONFINITE
    p, st = orc.softmax(np.array([-np.inf, 0.0], dtype=np.float32))
    assert st == 0 and p.tolist() == [0.0, 1.0]


# --------------------------------------------------------------------------- #
# inverse CDF
# --------------------------------------------------------------------------- #
def test_inverse_cdf_dyadic_boundaries():
    w = [0.5, 0.0, 0.25, 0.125, 0.125]
    cdf_edges = [(0.0, 0), (0.49999, 0), (0.5, 2), (0.74999, 2), (0.75, 3), (0.875, 4), (0.999999, 4)]
    for u, tok in cdf_edges:
        assert orc.sample(w, u)[0] == tok
    # unnormalised weights give the same answer
    for u, tok in cdf_edges:
        assert orc.sample([8 * x for x in w], u)[0] == tok
    # u = 0 selects the first token with positive weight
    assert orc.sample([0.0, 0.0, 1.0, 1.0], 0.0)[0] == 2
    # no mass at all
    assert orc.sample([0.0, 0.0], 0.3)[0] == -1


def test_inverse_cdf_measure_matches_weights():
    rng = np.random.default_rng(7)
    w = rng.random(7)
    w[3] = 0.0
    G = 20000
    counts = np.zeros(7)
    for j in range(G):
        counts[orc.sample(w, (j + 0.5) / G)[0]] += 1
    assert np.allclose(counts / G, w / w.sum(), atol=1.5 / G)
    assert counts[3] == 0


def test_inverse_cdf_margin_and_band():
    w = [0.25, 0.25, 0.5]
    tok, lo, hi, mg = orc.sample(w, 0.3, band=1e-3)
    assert (tok, lo, hi) == (1, 1, 1) and mg == pytest.approx(0.05, abs=1e-15)
    tok, lo, hi, mg = orc.sample(w, 0.2501, band=1e-3)
    assert (tok, lo, hi) == (1, 0, 1) and mg == pytest.approx(1e-4, abs=1e-12)
    tok, lo, hi, mg = orc.sample(w, 0.4995, band=1e-3)
    assert (tok, lo, hi) == (1, 1, 2)


def test_argmax_ties_to_lowest_index():
    assert orc.argmax([0.1, 0.4, 0.4, 0.1]) == 1
    assert orc.argmax([0.0, 0.0]) == -1


# --------------------------------------------------------------------------- #
# chain logic
# --------------------------------------------------------------------------- #
def _small_chain(seed=0, B=3, gamma=4, V=11, identical_at=()):
    rng = np.random.default_rng(seed)
    target = (rng.normal(size=(B, gamma + 1, V)) * 2).astype(np.float32)
    draft = (target[:, :gamma] + rng.normal(size=(B, gamma, V)) * rng.random((B, gamma, 1)) * 2).astype(np.float32)
    for (b, i) in identical_at:
        draft[b, i] = target[b, i]
    tokens = rng.integers(0, V, size=(B, gamma)).astype(np.int32)
    ua = rng.random((B, gamma)).astype(np.float32)
    us = rng.random(B).astype(np.float32)
    return target, draft, tokens, ua, us


def test_threshold_extremes_and_monotonicity():
    target, draft, tokens, ua, us = _small_chain(1)
    B, gamma = tokens.shape
    base = orc.verify_chain(target, draft, tokens, ua, us, dtype="f32", T=0.5)
    D = base.divergence
    lo = orc.verify_chain(target, draft, None, None, us, dtype="f32", T=D.min() * 0.5)
    assert (lo.accept_len == 0).all()
    hi = orc.verify_chain(target, draft, None, None, us, dtype="f32", T=D.max() * 1.01)
    assert (hi.accept_len == gamma).all()
    # bonus token comes from the row after the last candidate
    for b in range(B):
        p, _ = orc.softmax(target[b, gamma])
        assert hi.next_token[b] == orc.sample(p, float(us[b]))[0]
        p0, _ = orc.softmax(target[b, 0])
        assert lo.next_token[b] == orc.sample(p0, float(us[b]))[0]
    prev = np.zeros(B, dtype=np.int32)
    for T in np.linspace(0.0, D.max() * 1.1, 40):
        r = orc.verify_chain(target, draft, None, None, us, dtype="f32", T=float(T))
        assert (r.accept_len >= prev).all()
        prev = r.accept_len
        # accept_len is the first position whose divergence fails the test
        for b in range(B):
            fails = [i for i in range(gamma) if not (D[b, i] < T)]
            assert r.accept_len[b] == (fails[0] if fails else gamma)


def test_fsd_ignores_tokens_and_accept_uniforms():
    target, draft, tokens, ua, us = _small_chain(2)
    r1 = orc.verify_chain(target, draft, tokens, ua, us, dtype="f32", T=0.3)
    r2 = orc.verify_chain(target, draft, (tokens + 3) % 11, 1.0 - ua, us, dtype="f32", T=0.3)
    r3 = orc.verify_chain(target, draft, None, None, us, dtype="f32", T=0.3)
    for r in (r2, r3):
        assert (r.accept_len == r1.accept_len).all() and (r.next_token == r1.next_token).all()
        assert (r.divergence == r1.divergence).all()


def test_strict_and_nonstrict_compare_differ_only_at_equality():
    target, draft, tokens, ua, us = _small_chain(3, identical_at=[(0, 0), (0, 1), (1, 0)])
    lt = orc.verify_chain(target, draft, None, None, us, dtype="f32", T=0.0, cmp="lt")
    le = orc.verify_chain(target, draft, None, None, us, dtype="f32", T=0.0, cmp="le")
    assert (lt.accept_len == 0).all()                       # Div < 0 never holds (Section 4.3)
    assert le.accept_len.tolist() == [2, 1, 0]              # only identical distributions pass at T = 0
    # T at the largest possible JS accepts everything under "<="
    a = np.array([[[0.0, -np.inf], [0.0, 0.0]]], dtype=np.float32)
    b = np.array([[[-np.inf, 0.0]]], dtype=np.float32)
    assert orc.verify_chain(a, b, None, None, us[:1], dtype="f32", T=LN2, cmp="le").accept_len[0] == 1
    assert orc.verify_chain(a, b, None, None, us[:1], dtype="f32", T=LN2, cmp="lt").accept_len[0] == 0


def test_forced_bits_override_decisions():
    target, draft, tokens, ua, us = _small_chain(4)
    forced = np.full(tokens.shape, -1, dtype=np.int8)
    forced[:, 0] = 1
    forced[:, 1] = 0
    r = orc.verify_chain(target, draft, None, None, us, dtype="f32", T=0.0, forced=forced)
    assert (r.accept_len == 1).all()


def test_hand_case_gamma2_v4():
    """gamma = 2, V = 4, worked by hand: position 0 identical (D = 0), position 1 is case C
    of the golden file (JS = 0.10644).  Target rows: p0 = p1 = (.1,.2,.3,.4); bonus row (1/2,1/4,1/8,1/8)."""
    p = [0.1, 0.2, 0.3, 0.4]
    q1 = [0.4, 0.3, 0.2, 0.1]
    bonus = [0.5, 0.25, 0.125, 0.125]
    target = np.stack([_logits_of(p), _logits_of(p), _logits_of(bonus)])[None]
    draft = np.stack([_logits_of(p), _logits_of(q1)])[None]
    us = np.array([0.55], dtype=np.float32)
    # T = 0.2: both pass -> n = 2, bonus token at u = .55 -> CDF (.5,.75,...) -> token 1
    r = orc.verify_chain(target, draft, None, None, us, dtype="f32", T=0.2)
    assert r.accept_len[0] == 2 and r.next_token[0] == 1
    assert r.divergence[0, 0] == 0.0 and r.divergence[0, 1] == pytest.approx(0.10644013528622315, abs=5e-7)
    # T = 0.1: position 1 fails -> n = 1, token from p at u = .55 -> CDF (.1,.3,.6,1) -> token 2
    r = orc.verify_chain(target, draft, None, None, us, dtype="f32", T=0.1)
    assert r.accept_len[0] == 1 and r.next_token[0] == 2
    # greedy on rejection (Section 6.3): argmax of p -> token 3
    r = orc.verify_chain(target, draft, None, None, us, dtype="f32", T=0.1, sample_kind="greedy")
    assert r.accept_len[0] == 1 and r.next_token[0] == 3
    # SD at position 1 with draft token 0: P_accept = min(1, .1/.4) = .25 (Eq. 1)
    toks = np.array([[2, 0]], dtype=np.int32)
    ua = np.array([[0.9, 0.2]], dtype=np.float32)      # position 0: ratio 1 > .9 accept; position 1: .25 > .2 accept
    r = orc.verify_chain(target, draft, toks, ua, us, dtype="f32", mode="sd")
    assert r.p_accept[0].tolist() == pytest.approx([1.0, 0.25], abs=1e-6) and r.accept_len[0] == 2
    ua = np.array([[0.9, 0.3]], dtype=np.float32)      # .25 > .3 fails -> residual max(0,p-q) = (0,0,.1,.3)/.4
    r = orc.verify_chain(target, draft, toks, ua, us, dtype="f32", mode="sd")
    assert r.accept_len[0] == 1 and r.next_token[0] == 3          # t = .55*.4 = .22 > .1 -> token 3
    us2 = np.array([0.2], dtype=np.float32)
    r = orc.verify_chain(target, draft, toks, ua, us2, dtype="f32", mode="sd")
    assert r.next_token[0] == 2                                    # t = .08 < .1 -> token 2
    r = orc.verify_chain(target, draft, toks, ua, us2, dtype="f32", mode="sd", sample_kind="greedy")
    assert r.next_token[0] == 3                                    # largest residual


# --------------------------------------------------------------------------- #
# SD mode: brute force on tiny vocabularies
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("V", [4, 5, 8])
def test_sd_preserves_target_distribution_bruteforce(V):
    """One candidate position.  Enumerate the draft token x ~ q and integrate both uniforms on a
    grid: the emitted token (x if accepted, else the resampled one) must be distributed as p, and
    the acceptance probability must be 1 - TV(p, q)."""
    rng = np.random.default_rng(100 + V)
    p = _rand_probs(rng, V)
    q = _rand_probs(rng, V)
    if V == 5:
        p[1] = 0.0
        p /= p.sum()
    G = 120
    grid = ((np.arange(G) + 0.5) / G).astype(np.float32)
    xs, uas, uss = np.meshgrid(np.arange(V), grid, grid, indexing="ij")
    Bn = xs.size
    target = np.broadcast_to(np.stack([_logits_of(p), _logits_of(p)]), (Bn, 2, V)).copy()
    draft = np.broadcast_to(_logits_of(q), (Bn, 1, V)).copy()
    r = orc.verify_chain(target, draft, xs.reshape(Bn, 1).astype(np.int32), uas.reshape(Bn, 1).astype(np.float32),
                         uss.reshape(Bn).astype(np.float32), dtype="f32", mode="sd")
    weight = q[xs.reshape(-1)] / (G * G)
    emitted = np.where(r.accept_len == 1, xs.reshape(-1), r.next_token)
    dist = np.bincount(emitted, weights=weight, minlength=V)
    assert np.allclose(dist, p, atol=2.5 / G)
    acc = weight[r.accept_len == 1].sum()
    assert acc == pytest.approx(1.0 - orc.divergence_probs(p, q, "tv"), abs=1.5 / G)


def test_sd_accept_prob_special_cases():
    assert orc.sd_accept_prob(0.2, 0.4) == 0.5
    assert orc.sd_accept_prob(0.4, 0.2) == 1.0
    assert orc.sd_accept_prob(0.1, 0.0) == 1.0
    assert orc.sd_accept_prob(0.0, 0.0) == 0.0
    # identical distributions: every candidate is accepted whatever the uniform
    target, draft, tokens, ua, us = _small_chain(5)
    draft = target[:, :-1].copy()
    r = orc.verify_chain(target, draft, tokens, ua, us, dtype="f32", mode="sd")
    assert (r.accept_len == tokens.shape[1]).all()


def test_rfsd_reduces_to_sd_at_zero_threshold():
    target, draft, tokens, ua, us = _small_chain(6, B=40)
    sd = orc.verify_chain(target, draft, tokens, ua, us, dtype="f32", mode="sd")
    rf = orc.verify_chain(target, draft, tokens, ua, us, dtype="f32", mode="rfsd", T=0.0, cmp="lt")
    assert (sd.accept_len == rf.accept_len).all() and (sd.next_token == rf.next_token).all()
    assert len(set(sd.accept_len.tolist())) > 1
    # with a positive threshold rFSD accepts at least as much as either rule alone (Eq. 6 is an OR)
    fsd = orc.verify_chain(target, draft, tokens, ua, us, dtype="f32", mode="fsd", T=0.15)
    rf2 = orc.verify_chain(target, draft, tokens, ua, us, dtype="f32", mode="rfsd", T=0.15)
    assert (rf2.accept_bits == (fsd.accept_bits | sd.accept_bits)).all()
    assert (rf2.accept_len >= np.maximum(fsd.accept_len, sd.accept_len)).all()


# --------------------------------------------------------------------------- #
# trees
# --------------------------------------------------------------------------- #
def _small_tree(seed, B, N, V, parent):
    rng = np.random.default_rng(seed)
    target = (rng.normal(size=(B, N + 1, V)) * 2).astype(np.float32)
    draft = np.empty((B, N, V), dtype=np.float32)
    for b in range(B):
        for j in range(N):
            draft[b, j] = target[b, parent[b, j] + 1] + rng.normal(size=V) * rng.random() * 1.5
    us = rng.random(B).astype(np.float32)
    return target, draft, us


def test_chain_shaped_tree_equals_chain_call():
    B, N, V = 5, 6, 13
    parent = np.tile(np.arange(-1, N - 1, dtype=np.int32), (B, 1))
    target, draft, us = _small_tree(11, B, N, V, parent)
    for T in (0.02, 0.1, 0.3, 1.0):
        c = orc.verify_chain(target, draft, None, None, us, dtype="f32", T=T)
        t = orc.verify_tree(target, draft, parent, us, max_depth=N, dtype="f32", T=T)
        assert (c.accept_len == t.accept_len).all() and (c.next_token == t.next_token).all()
        assert (c.divergence == t.divergence).all()
        for b in range(B):
            n = int(t.accept_len[b])
            assert t.path[b, :n].tolist() == list(range(n)) and (t.path[b, n:] == -1).all()


def test_star_tree_picks_lowest_passing_child():
    B, N, V = 6, 3, 9
    parent = np.full((B, N), -1, dtype=np.int32)
    target, draft, us = _small_tree(12, B, N, V, parent)
    seen = set()
    for T in (0.01, 0.03, 0.12):
        r = orc.verify_tree(target, draft, parent, us, max_depth=3, dtype="f32", T=T)
        for b in range(B):
            passing = [j for j in range(N) if r.divergence[b, j] < T]
            assert r.accept_len[b] == (1 if passing else 0)
            assert r.end_node[b] == (passing[0] if passing else -1)
            seen.add(int(r.end_node[b]))
            # every node is compared with the root's target row
            for j in range(N):
                assert r.divergence[b, j] == orc.divergence_logits(target[b, 0], draft[b, j], "js")
    assert -1 in seen and len(seen) >= 3


def test_tree_bruteforce_paths():
    rng = np.random.default_rng(13)
    for trial in range(30):
        N = int(rng.integers(2, 10))
        parent = np.array([[int(rng.integers(-1, j)) for j in range(N)]], dtype=np.int32)
        target, draft, us = _small_tree(1000 + trial, 1, N, 7, parent)
        T = float(rng.choice([0.05, 0.15, 0.4]))
        max_depth = int(rng.integers(1, 5))
        r = orc.verify_tree(target, draft, parent, us, max_depth=max_depth, dtype="f32", T=T)
        # independent enumeration: for every node walk up to the root
        best, best_depth = -1, 0
        for j in range(N):
            chain = []
            k = j
            while k >= 0:
                chain.append(k)
                k = int(parent[0, k])
            ok = all(orc.divergence_logits(target[0, parent[0, k] + 1], draft[0, k], "js") < T for k in chain)
            if ok and len(chain) <= max_depth and len(chain) > best_depth:
                best, best_depth = j, len(chain)
        assert r.end_node[0] == best and r.accept_len[0] == best_depth
        expect_path = []
        k = best
        while k >= 0:
            expect_path.append(k)
            k = int(parent[0, k])
        expect_path = expect_path[::-1] + [-1] * (max_depth - best_depth)
        assert r.path[0].tolist() == expect_path
        p, _ = orc.softmax(target[0, best + 1])
        assert r.next_token[0] == orc.sample(p, float(us[0]))[0]


def test_bad_tree_is_flagged():
    parent = np.array([[-1, 0, 2, 1]], dtype=np.int32)      # node 2 names itself as parent
    target, draft, us = _small_tree(14, 1, 4, 5, np.array([[-1, 0, 1, 1]]))
    r = orc.verify_tree(target, draft, parent, us, max_depth=4, dtype="f32", T=10.0)
    assert r.row_status[0] & orc.ST_BADTREE and r.accept_len[0] == 0 and r.next_token[0] == -1
    assert (r.path[0] == -1).all()


def test_nonfinite_position_is_rejected_and_flagged():
    target, draft, tokens, ua, us = _small_chain(8, B=2)
    draft[1, 1, 3] = np.nan
    r = orc.verify_chain(target, draft, tokens, ua, us, dtype="f32", T=100.0)
    assert r.accept_len.tolist() == [4, 1]
    assert r.row_status.tolist() == [0, orc.ST_NONFINITE]
    assert np.isnan(r.divergence[1, 1])
    p, _ = orc.softmax(target[1, 1])
    assert r.next_token[1] == orc.sample(p, float(us[1]))[0]


# --------------------------------------------------------------------------- #
# edge rules of the token draw and of the ratio test, each worked by hand
# --------------------------------------------------------------------------- #
def test_residual_without_mass_falls_back_to_the_target_distribution():
    """Eq. 3 with P_T == P_D: max(0, P_T - P_D) has no mass, so the replacement comes from P_T.
    The rejection is forced by a draft token outside the vocabulary.  P_T = (1/2,1/4,1/8,1/8):
    CDF (.5,.75,.875,1) -> u = .6 gives token 1, u = .8 gives token 2, u = .9 gives token 3."""
    p = [0.5, 0.25, 0.125, 0.125]
    target = np.stack([_logits_of(p), _logits_of([0.25] * 4)])[None]
    draft = _logits_of(p)[None, None]
    toks = np.array([[4]], dtype=np.int32)
    ua = np.zeros((1, 1), dtype=np.float32)
    for u, want in ((0.6, 1), (0.8, 2), (0.9, 3), (0.0, 0)):
        for mode in ("sd", "rfsd"):
            r = orc.verify_chain(target, draft, toks, ua, np.array([u], np.float32), dtype="f32", mode=mode,
                                 T=0.0, cmp="lt")
            assert r.accept_len[0] == 0 and r.next_token[0] == want and r.row_status[0] == 0
    r = orc.verify_chain(target, draft, toks, ua, np.array([0.9], np.float32), dtype="f32", mode="sd",
                         sample_kind="greedy")
    assert r.next_token[0] == 0                                   # argmax of P_T, not of an empty residual


def test_rejection_on_a_nonfinite_draft_row_draws_from_the_target_distribution():
    """SD mode, draft row with a NaN: the position is rejected and flagged, and since no residual
    can be formed the token comes from P_T = (1/8,1/8,1/4,1/2): CDF (.125,.25,.5,1)."""
    p = [0.125, 0.125, 0.25, 0.5]
    target = np.stack([_logits_of(p), _logits_of([0.25] * 4)])[None]
    draft = _logits_of([0.7, 0.1, 0.1, 0.1])[None, None].copy()
    draft[0, 0, 1] = np.nan
    toks = np.array([[3]], dtype=np.int32)
    ua = np.zeros((1, 1), dtype=np.float32)
    for u, want in ((0.05, 0), (0.2, 1), (0.3, 2), (0.7, 3)):
        for mode in ("sd", "rfsd"):
            r = orc.verify_chain(target, draft, toks, ua, np.array([u], np.float32), dtype="f32", mode=mode, T=5.0)
            assert r.accept_len[0] == 0 and r.row_status[0] == orc.ST_NONFINITE
            assert r.next_token[0] == want
    # the same with the draft row +inf at the would-be residual's favourite token
    draft[0, 0, 1] = np.inf
    r = orc.verify_chain(target, draft, toks, ua, np.array([0.3], np.float32), dtype="f32", mode="sd")
    assert r.accept_len[0] == 0 and r.next_token[0] == 2 and r.row_status[0] == orc.ST_NONFINITE


def test_token_ids_outside_the_vocabulary_fail_the_ratio_test():
    """Eq. 1-2 need P(x) of a token of the vocabulary: ids -1 and V never pass the ratio test,
    whatever the uniform; under Eq. 6 such a position passes only through Div < T.
    Position rows: p = (.1,.2,.3,.4), q = (.4,.3,.2,.1) -> JS = 0.10644 (golden case C)."""
    p, q = [0.1, 0.2, 0.3, 0.4], [0.4, 0.3, 0.2, 0.1]
    V = 4
    target = np.stack([_logits_of(p)] * 3)[None].repeat(3, axis=0)          # [3, 3, V]
    draft = np.stack([_logits_of(q)] * 2)[None].repeat(3, axis=0)           # [3, 2, V]
    toks = np.array([[-1, 3], [3, V], [3, 3]], dtype=np.int32)              # token 3: ratio .4/.1 -> P_accept = 1
    ua = np.zeros((3, 2), dtype=np.float32)                                 # u = 0: every in-range token passes
    us = np.full(3, 0.5, dtype=np.float32)
    r = orc.verify_chain(target, draft, toks, ua, us, dtype="f32", mode="sd")
    assert r.accept_len.tolist() == [0, 1, 2]
    assert r.accept_bits.tolist() == [[0, 1], [1, 0], [1, 1]]
    assert np.isnan(r.p_accept[0, 0]) and np.isnan(r.p_accept[1, 1])
    # rFSD below the divergence: the same; above it: the divergence rule accepts them
    r = orc.verify_chain(target, draft, toks, ua, us, dtype="f32", mode="rfsd", T=0.1)
    assert r.accept_len.tolist() == [0, 1, 2]
    r = orc.verify_chain(target, draft, toks, ua, us, dtype="f32", mode="rfsd", T=0.11)
    assert r.accept_len.tolist() == [2, 2, 2]
    # a rejected out-of-range token is replaced from the residual max(0, p - q) = (0,0,.1,.3)/.4:
    # t = .5 * .4 = .2 > .1 -> token 3
    r = orc.verify_chain(target, draft, toks, ua, us, dtype="f32", mode="sd")
    assert r.next_token[0] == 3 and r.next_token[1] == 3


def test_inverse_cdf_without_a_crossing_takes_the_last_token_that_has_weight():
    """u * W at or above the last cumulative sum (u = 1, or rounding): the largest k with
    w_k > 0, not the last index."""
    w = [0.25, 0.5, 0.25, 0.0, 0.0]
    assert orc.sample(w, 1.0)[0] == 2
    assert orc.sample(w, float(np.nextafter(np.float32(1), np.float32(0))))[0] == 2
    assert orc.sample([0.0, 3.0, 0.0], 1.0)[0] == 1
    assert orc.sample([0.0, 3.0, 0.0], 0.0)[0] == 1               # zero-weight entries are never chosen
    # band edges past the total mass clamp to the same rule
    tok, lo, hi, _ = orc.sample(w, 1.0 - 1e-9, band=1e-6)
    assert (tok, lo, hi) == (2, 2, 2)
    # through the chain call: a target row whose trailing entries are masked, u as close to 1 as fp32 allows
    a = _logits_of([0.25, 0.5, 0.25, 0.0, 0.0])
    target = np.stack([a, a])[None]
    draft = _logits_of([0.2] * 5)[None, None]
    us = np.array([np.nextafter(np.float32(1), np.float32(0))], dtype=np.float32)
    r = orc.verify_chain(target, draft, None, None, us, dtype="f32", T=0.0, cmp="lt")
    assert r.accept_len[0] == 0 and r.next_token[0] == 2
