"""fsd_verify_chain_static: the entry point for callers that cannot hand the library any scratch
memory (their device memory was all assigned at start-up, or they run inside another framework's
allocator and may not call cudaMalloc themselves).  It must give the same outputs as
fsd_verify_chain, call after call, although all calls share one scratch array that keeps the
previous call's contents.  This file is named to be collected last."""

import numpy as np
import pytest
import torch

import fsd_inputs as gi
import paper_2502_20704_b200 as fsd
from paper_2502_20704_b200 import binding


def _outputs(B, gamma):
    return (torch.full((B,), -9, dtype=torch.int32, device="cuda"),
            torch.full((B,), -9, dtype=torch.int32, device="cuda"),
            torch.full((B, gamma), -9.0, dtype=torch.float32, device="cuda"),
            torch.full((B,), -9, dtype=torch.int32, device="cuda"))


def _dev(a):
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


@pytest.mark.gpu
def test_static_scratch_entry_matches_workspace_entry_on_consecutive_calls():
    stream = torch.cuda.current_stream().cuda_stream
    # two different batches back to back: the second call finds the first call's leftovers in the
    # shared array; a third call repeats the first batch with another rule
    calls = [
        (gi.make_chain(6, 5, 32000, dtype="bf16", recipe="zipf", sigma=(0.2, 1.5), sigma_mode="uniform",
                       workload_id=700), dict(mode="fsd", T=0.1)),
        (gi.make_chain(3, 7, 4099, dtype="f32", recipe="spike", sigma=(0.3, 1.0), workload_id=701),
         dict(mode="sd", T=0.0)),
        (gi.make_chain(6, 5, 32000, dtype="bf16", recipe="zipf", sigma=(0.2, 1.5), sigma_mode="uniform",
                       workload_id=700), dict(mode="rfsd", T=0.05, div="tv")),
    ]
    for c, kw in calls:
        opts = fsd.make_opts(dtype=c.dtype, **kw)
        t, d = _dev(c.target), _dev(c.draft)
        tok, ua, us = _dev(c.draft_tokens), _dev(c.u_accept), _dev(c.u_sample)
        ref = _outputs(c.B, c.gamma)
        wsb = fsd.fsd_workspace_bytes(c.B, c.gamma, c.V, opts)
        ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
        rc = fsd.fsd_verify_chain(t, d, tok, ua, us, c.B, c.gamma, c.V, opts, *ref, ws, wsb, stream)
        assert rc == 0, fsd.fsd_status_string(rc)
        got = _outputs(c.B, c.gamma)
        rc = fsd.fsd_verify_chain_static(t, d, tok, ua, us, c.B, c.gamma, c.V, opts, *got, stream)
        assert rc == 0, fsd.fsd_status_string(rc)
        torch.cuda.synchronize()
        for name, r, g in zip(("accept_len", "next_token", "divergence", "row_status"), ref, got):
            r, g = r.cpu().numpy(), g.cpu().numpy()
            if name == "divergence":
                # same kernels, same inputs, same reduction order: the same bits
                assert np.array_equal(g.view(np.uint32), r.view(np.uint32)), name
            else:
                assert np.array_equal(g, r), name
        assert (got[0].cpu().numpy() >= 0).all()


def test_static_scratch_entry_refuses_oversized_calls():
    # refused on the host before anything touches a device, so this part needs no GPU
    o = fsd.make_opts(T=0.2)
    big_B = binding.FSD_STATIC_MAX_POSITIONS // 8 + 1
    rc = fsd.fsd_verify_chain_static(4096, 4096, None, None, 4096, big_B, 8, 64, o, 4096, 4096, 4096, 4096, None)
    assert rc == binding.FSD_ERR_TOO_LARGE
    assert "FSD_STATIC_MAX_POSITIONS" in fsd.fsd_status_string(rc)
    assert fsd.fsd_verify_chain_static(None, 4096, None, None, 4096, 2, 8, 64, o, 4096, 4096, 4096, 4096,
                                       None) == binding.FSD_ERR_NULL
