"""GPU-vs-oracle parity on seeded random shapes, dtypes, divergences, modes and thresholds.

The named workloads fix a handful of shapes; this sweep draws others (vocabulary sizes that are
and are not multiples of the vector width, group sizes 1 to 16, one to five ring stages per
pair, masked entries) so that every launch configuration of the pair kernels meets the oracle.
The number of cases is small by default; FSD_SWEEP_CASES and FSD_SD_SWEEP_CASES in the environment
extend the two chain sweeps (every case is seeded by its index, so a longer sweep repeats the
shorter one and goes on).
"""

import os

import numpy as np
import pytest

import fsd_inputs as gi
from tests import parity

pytestmark = pytest.mark.gpu


def _case(it: int):
    rng = np.random.default_rng(20704 + it)
    dtype = str(rng.choice(["bf16", "f32"]))
    V = int(rng.choice([8 * rng.integers(8, 400), 8 * rng.integers(400, 6000), 8 * rng.integers(6000, 20000),
                        int(rng.integers(9, 5000))]))
    B, gamma = int(rng.integers(1, 40)), int(rng.integers(1, 12))
    if B * gamma * V > 3e7:
        B = max(1, int(3e7 / (gamma * V)))
    opts = dict(div=str(rng.choice(["js", "kl", "tv"])), mode=str(rng.choice(["fsd", "fsd", "sd", "rfsd"])),
                sample=str(rng.choice(["invcdf", "invcdf", "greedy"])), cmp=str(rng.choice(["lt", "le"])),
                T=float(rng.choice([0.0, 0.02, 0.1, 0.3, 0.7, 2.0])))
    recipe = str(rng.choice(["spike", "zipf"]))
    c = gi.make_chain(B, gamma, V, dtype=dtype, recipe=recipe, sigma=(0.1, 2.0), sigma_mode="uniform",
                      disjoint_frac=0.1 if recipe == "zipf" else 0.0, workload_id=2000 + it)
    if rng.random() < 0.3:                          # masked vocabulary entries (same mask in every row)
        f32 = dtype == "f32"
        t = c.target if f32 else gi.bf16_bits_to_f32(c.target)
        d = c.draft if f32 else gi.bf16_bits_to_f32(c.draft)
        t[:, :, rng.random(V) < 0.3] = -np.inf
        if rng.random() < 0.5:
            d[:, :, rng.random(V) < 0.2] = -np.inf
        if not f32:
            c.target[:] = gi.f32_to_bf16_bits(t)
            c.draft[:] = gi.f32_to_bf16_bits(d)
    return c, opts


@pytest.mark.parametrize("it", range(int(os.environ.get("FSD_SWEEP_CASES", "24"))))
def test_random_shape_matches_oracle(it):
    c, opts = _case(it)
    r = parity.check_chain(c.target, c.draft, c.draft_tokens, c.u_accept, c.u_sample, c.dtype, **opts)
    assert r["max_err"] < (1e-5 if c.dtype == "f32" else 1e-4)


@pytest.mark.parametrize("it", range(8))
def test_random_tree_matches_oracle(it):
    rng = np.random.default_rng(40704 + it)
    dtype = str(rng.choice(["bf16", "f32"]))
    V = int(rng.choice([8 * rng.integers(16, 600), 8 * rng.integers(600, 9000), int(rng.integers(9, 3000))]))
    B, N = int(rng.integers(1, 9)), int(rng.integers(1, 40))
    depth, children = int(rng.integers(1, 8)), int(rng.integers(1, 5))
    N = min(N, sum(children ** d for d in range(1, depth + 1)))      # what the limits can hold
    if B * N * V > 2e7:
        B = max(1, int(2e7 / (N * V)))
    t = gi.make_tree(B, N, V, dtype=dtype, recipe=str(rng.choice(["spike", "zipf"])), sigma=float(rng.uniform(0.2, 1.5)),
                     max_depth=depth, max_children=children, workload_id=3000 + it)
    parity.check_tree(t, T=float(rng.choice([0.02, 0.1, 0.3, 0.7])), div=str(rng.choice(["js", "kl", "tv"])),
                      cmp=str(rng.choice(["lt", "le"])), sample=str(rng.choice(["invcdf", "greedy"])))


@pytest.mark.parametrize("it", range(int(os.environ.get("FSD_SD_SWEEP_CASES", "12"))))
def test_random_sd_and_rfsd_draws_match_oracle(it):
    """SD and rFSD only, on larger vocabularies: the residual draw in its one-pass and two-pass forms."""
    rng = np.random.default_rng(99000 + it)
    V = int(8 * rng.integers(500, 20000))
    B, gamma = int(rng.integers(1, 12)), int(rng.integers(1, 8))
    dtype, recipe = str(rng.choice(["bf16", "f32"])), str(rng.choice(["spike", "zipf"]))
    c = gi.make_chain(B, gamma, V, dtype=dtype, recipe=recipe, sigma=(0.05, 2.0), sigma_mode="uniform",
                      disjoint_frac=0.1 if recipe == "zipf" else 0.0, workload_id=7000 + it)
    parity.check_chain(c.target, c.draft, c.draft_tokens, c.u_accept, c.u_sample, c.dtype, mode=str(rng.choice(["sd", "rfsd"])),
                       T=float(rng.choice([0.0, 0.05, 0.3])), sample=str(rng.choice(["invcdf", "invcdf", "greedy"])))

