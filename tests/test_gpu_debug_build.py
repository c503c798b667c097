"""The debug build of the library (the same kernels with their index and range checks compiled
in) run on chain, tree, fp32, ragged and non-vector shapes in a process of its own: results must
still match the oracle and the workspace's debug word must stay zero."""

import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

pytestmark = pytest.mark.gpu

_SCRIPT = r"""
import numpy as np, torch
import fsd_inputs as gi
import paper_2502_20704_b200 as fsd
from tests import parity

assert fsd.fsd_debug_checks()[0], "this process must have loaded the debug build"
words = []
orig_empty = torch.empty

def run(c, tree=False, **kw):
    # parity.* allocate the workspace themselves: read the debug word back through a wrapper
    B = c.B
    P = c.N if tree else c.gamma
    _, off = fsd.fsd_debug_checks(B, P)
    seen = {}
    def spy(*a, **k):
        t = orig_empty(*a, **k)
        if k.get("dtype") == torch.uint8 and k.get("device") == "cuda":
            seen["ws"] = t
        return t
    torch.empty = spy
    try:
        if tree:
            parity.check_tree(c, **kw)
        else:
            parity.check_chain(c.target, c.draft, c.draft_tokens, c.u_accept, c.u_sample, c.dtype, **kw)
    finally:
        torch.empty = orig_empty
    word = int(seen["ws"][off:off + 4].view(torch.int32).item())
    words.append(word)
    assert word == 0, f"range check failed: bits {word:#x}"

run(gi.make_chain(6, 5, 36000, dtype="bf16", recipe="zipf", sigma=(0.3, 1.5), sigma_mode="uniform", workload_id=440), T=0.2)
run(gi.make_chain(6, 5, 36000, dtype="bf16", recipe="zipf", sigma=(0.3, 1.5), sigma_mode="uniform", workload_id=440), T=0.2, mode="sd")
run(gi.make_chain(3, 4, 152064, dtype="bf16", recipe="zipf", sigma=(0.2, 2.0), sigma_mode="uniform", workload_id=441), T=0.2, div="tv")
run(gi.make_chain(3, 3, 32776, dtype="bf16", recipe="zipf", sigma=(0.5,), workload_id=442), T=0.1, div="kl")
run(gi.make_chain(2, 3, 100000, dtype="f32", recipe="spike", sigma=(0.5,), workload_id=443), T=0.1)
run(gi.make_chain(3, 2, 4099, dtype="f32", recipe="spike", sigma=(0.3, 1.0), workload_id=444), T=0.1, mode="rfsd")
run(gi.make_tree(3, 40, 32000, dtype="bf16", sigma=0.6, max_depth=5, workload_id=445), tree=True, T=0.05)
print("debug words", words)
"""


def test_debug_build_finds_no_range_violation_and_matches_the_oracle():
    from paper_2502_20704_b200 import build as lib_build
    lib = lib_build.build(debug=True)
    env = dict(os.environ, FSD_VERIFY_LIB=lib, PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    r = subprocess.run([sys.executable, "-c", _SCRIPT], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "debug words" in r.stdout
