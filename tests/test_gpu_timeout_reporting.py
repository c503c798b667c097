"""A device-side wait that runs out.  Two injections, neither of which faults or hangs anything:
the library raises the flag itself on the host side of the call (the reporting path alone), and
one thread block of the streaming kernel withholds a statistics message while the exchange wait's
limit is lowered to about a tenth of a second, so that the wait of its partners really runs out
and the kernel's own give-up path runs.  Either way the call must return, mark every row, and
leave the next call untouched."""

import numpy as np
import pytest

import fsd_inputs as gi
import paper_2502_20704_b200 as fsd
from paper_2502_20704_b200 import binding
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", [1, 2])
def test_injected_timeout_marks_every_row_and_the_next_call_is_clean(mode):
    c = gi.make_chain(6, 4, 36000, dtype="bf16", recipe="zipf", sigma=(0.3, 1.5), sigma_mode="uniform", workload_id=430)
    before = parity.check_chain(c.target, c.draft, c.draft_tokens, c.u_accept, c.u_sample, c.dtype, T=0.2)["gpu"]
    assert not (before.row_status & binding.FSD_ROW_TIMEOUT).any()
    assert fsd.fsd_set_timeout_injection(mode) == 0
    try:
        marked = parity.run_chain_gpu(c.target, c.draft, None, None, c.u_sample, c.dtype, T=0.2)
    finally:
        fsd.fsd_set_timeout_injection(0)
    assert (marked.row_status & binding.FSD_ROW_TIMEOUT).all()          # the call returned and says so in every row
    after = parity.run_chain_gpu(c.target, c.draft, None, None, c.u_sample, c.dtype, T=0.2)
    assert np.array_equal(after.row_status, before.row_status)
    assert np.array_equal(after.accept_len, before.accept_len) and np.array_equal(after.next_token, before.next_token)
    assert np.array_equal(after.divergence.view(np.uint32), before.divergence.view(np.uint32))


def test_a_wait_that_runs_out_in_a_call_that_fills_the_gpu():
    """512 pairs on all SMs, one group's exchange runs out: the groups that see the flag take no
    further pairs, the call returns marked, and the next call is right."""
    c = gi.make_chain(64, 8, 32000, dtype="bf16", recipe="spike", sigma=(0.3, 1.0), sigma_mode="uniform", workload_id=431)
    assert fsd.fsd_set_timeout_injection(2) == 0
    try:
        marked = parity.run_chain_gpu(c.target, c.draft, None, None, c.u_sample, c.dtype, T=0.2)
    finally:
        fsd.fsd_set_timeout_injection(0)
    assert (marked.row_status & binding.FSD_ROW_TIMEOUT).all()
    parity.check_chain(c.target, c.draft, c.draft_tokens, c.u_accept, c.u_sample, c.dtype, T=0.2)
    assert fsd.fsd_set_timeout_injection(3) != 0
