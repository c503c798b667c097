"""The reporting path of a device-side wait that ran out, exercised without making a GPU wait for
something that never comes: the library is told to raise the flag itself (on the host side of
the call), and the call must return, mark every row, and leave the next call untouched."""

import numpy as np
import pytest

import fsd_inputs as gi
import paper_2502_20704_b200 as fsd
from paper_2502_20704_b200 import binding
from tests import parity

pytestmark = pytest.mark.gpu


def test_injected_timeout_marks_every_row_and_the_next_call_is_clean():
    c = gi.make_chain(6, 4, 36000, dtype="bf16", recipe="zipf", sigma=(0.3, 1.5), sigma_mode="uniform", workload_id=430)
    before = parity.check_chain(c.target, c.draft, c.draft_tokens, c.u_accept, c.u_sample, c.dtype, T=0.2)["gpu"]
    assert not (before.row_status & binding.FSD_ROW_TIMEOUT).any()
    fsd.fsd_set_timeout_injection(True)
    try:
        marked = parity.run_chain_gpu(c.target, c.draft, None, None, c.u_sample, c.dtype, T=0.2)
    finally:
        fsd.fsd_set_timeout_injection(False)
    assert (marked.row_status & binding.FSD_ROW_TIMEOUT).all()          # the call returned and says so in every row
    after = parity.run_chain_gpu(c.target, c.draft, None, None, c.u_sample, c.dtype, T=0.2)
    assert np.array_equal(after.row_status, before.row_status)
    assert np.array_equal(after.accept_len, before.accept_len) and np.array_equal(after.next_token, before.next_token)
    assert np.array_equal(after.divergence.view(np.uint32), before.divergence.view(np.uint32))
