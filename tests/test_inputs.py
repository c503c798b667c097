"""The seeded input generators: determinism, shapes, value ranges, tree structure."""

import numpy as np

import fsd_inputs as gi


def test_bf16_round_trip_and_rounding():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 0.0, np.inf, -np.inf, 3.0e38], dtype=np.float32)
    bits = gi.f32_to_bf16_bits(x)
    back = gi.bf16_bits_to_f32(bits)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7: ties go to the even mantissa (1.0)
    assert back[0] == 1.0 and back[1] == 1.0
    # 1 + 3*2^-8 is a tie between 1 + 2^-7 (odd) and 1 + 2^-6 (even)
    assert back[2] == np.float32(1.015625)
    assert back[3] == -2.5 and back[4] == 0.0 and back[5] == np.inf and back[6] == -np.inf
    assert np.isfinite(back[7])
    assert np.isnan(gi.bf16_bits_to_f32(gi.f32_to_bf16_bits(np.array([np.nan], np.float32)))[0])
    r = np.random.default_rng(0).normal(size=1000).astype(np.float32) * 10
    err = np.abs(gi.bf16_bits_to_f32(gi.f32_to_bf16_bits(r)) - r)
    assert (err <= np.abs(r) * 2.0 ** -8).all()


def test_chain_is_deterministic_and_well_formed():
    a = gi.make_chain(3, 4, 512, dtype="bf16", recipe="zipf", sigma=(0.2, 2.0), sigma_mode="uniform",
                      disjoint_frac=0.3, workload_id=77)
    b = gi.make_chain(3, 4, 512, dtype="bf16", recipe="zipf", sigma=(0.2, 2.0), sigma_mode="uniform",
                      disjoint_frac=0.3, workload_id=77)
    for f in ("target", "draft", "draft_tokens", "u_accept", "u_sample", "sigma", "disjoint"):
        assert np.array_equal(getattr(a, f), getattr(b, f))
    assert a.target.shape == (3, 5, 512) and a.target.dtype == np.uint16
    assert a.draft.shape == (3, 4, 512)
    assert a.draft_tokens.dtype == np.int32 and (a.draft_tokens >= 0).all() and (a.draft_tokens < 512).all()
    assert a.u_accept.dtype == np.float32 and (a.u_accept >= 0).all() and (a.u_accept < 1).all()
    assert (a.sigma >= 0.2).all() and (a.sigma <= 2.0).all()
    assert a.ideal_bytes == 2 * 3 * 9 * 512
    c = gi.make_chain(3, 4, 512, dtype="bf16", recipe="zipf", workload_id=78)
    assert not np.array_equal(a.target, c.target)
    # a larger batch extends a smaller one row for row
    d = gi.make_chain(2, 4, 512, dtype="bf16", recipe="zipf", sigma=(0.2, 2.0), sigma_mode="uniform",
                      disjoint_frac=0.3, workload_id=77)
    assert np.array_equal(d.target, a.target[:2]) and np.array_equal(d.draft, a.draft[:2])


def test_spike_recipe_and_f32_storage():
    c = gi.make_chain(1, 3, 4096, dtype="f32", recipe="spike", sigma=(0.1, 0.5, 2.0), workload_id=5)
    assert c.target.dtype == np.float32
    assert c.sigma[0].tolist() == [0.1, 0.5, 2.0]
    assert abs(float(c.target.std()) - 3.0) < 0.1
    for i in range(3):
        noise = c.draft[0, i] - c.target[0, i]
        assert abs(float(noise.std()) - c.sigma[0, i]) < 0.1 * c.sigma[0, i]


def test_tree_structure_limits():
    t = gi.make_tree(4, 60, 256, max_depth=6, max_children=4, workload_id=9)
    assert t.parent.shape == (4, 60) and t.target.shape == (4, 61, 256) and t.draft.shape == (4, 60, 256)
    assert len({tuple(p) for p in t.parent.tolist()}) == 4
    for b in range(4):
        depth = {}
        kids = {}
        for j, p in enumerate(t.parent[b].tolist()):
            assert -1 <= p < j
            depth[j] = 1 if p < 0 else depth[p] + 1
            kids[p] = kids.get(p, 0) + 1
        assert max(depth.values()) <= 6 and max(kids.values()) <= 4


def test_named_configs_have_the_stated_shapes():
    want = {"c1": (1, 4, 32000, "f32"), "c2": (16, 5, 32000, "bf16"), "c3": (32, 6, 128256, "bf16"),
            "c4": (64, 8, 152064, "bf16")}
    for name, (B, g, V, dt) in want.items():
        p = gi.CONFIGS[name].params
        assert (p["B"], p["gamma"], p["V"], p["dtype"]) == (B, g, V, dt)
    p = gi.CONFIGS["c5"].params
    assert (p["B"], p["N"], p["V"], p["dtype"], p["max_depth"], p["max_children"]) == (8, 60, 32000, "bf16", 6, 4)
    c = gi.make_config("c4", B=1, gamma=2)
    assert c.target.shape == (1, 3, 152064)


def test_tree_unique_rows():
    parent = np.array([[-1, 0, 0, 1]], dtype=np.int32)
    # draft rows 4; parent contexts {root, node0, node1} = 3; end node 3 adds its own row
    assert gi.tree_unique_rows(parent, np.array([3])) == 4 + 4
    assert gi.tree_unique_rows(parent, np.array([1])) == 4 + 3
    assert gi.tree_unique_rows(parent, np.array([-1])) == 4 + 3
