"""GPU threshold-tuning helpers against the tuning oracle, through the C ABI: bit-exact."""

import numpy as np
import pytest

from oracle import fsd_tuning_oracle as tun

pytestmark = pytest.mark.gpu
F = np.float32
CMP = {"lt": 0, "le": 1}


def _dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _gpu_sweep(D, Ts, cmp):
    import torch
    import paper_2502_20704_b200 as fsd
    B, G = D.shape
    d, t = _dev(D), _dev(np.asarray(Ts, dtype=F))
    m = torch.full((len(Ts),), -1.0, device="cuda")
    f = torch.full((len(Ts),), -1.0, device="cuda")
    assert fsd.fsd_threshold_sweep(d, B, G, t, len(Ts), CMP[cmp], m, f, torch.cuda.current_stream().cuda_stream) == 0
    torch.cuda.synchronize()
    return m.cpu().numpy(), f.cpu().numpy()


def _gpu_calibrate(D, target, cmp):
    import torch
    import paper_2502_20704_b200 as fsd
    B, G = D.shape
    d = _dev(D)
    out = torch.full((2,), -1.0, device="cuda")
    assert fsd.fsd_calibrate_threshold(d, B, G, float(target), CMP[cmp], out[0:1], out[1:2],
                                       torch.cuda.current_stream().cuda_stream) == 0
    torch.cuda.synchronize()
    o = out.cpu().numpy()
    return o[0], o[1]


def _gpu_labels(D, T, cmp):
    import torch
    import paper_2502_20704_b200 as fsd
    B, G = D.shape
    d = _dev(D)
    lab = torch.full((B, G), 7, dtype=torch.uint8, device="cuda")
    assert fsd.fsd_accept_labels(d, B, G, float(T), CMP[cmp], lab, torch.cuda.current_stream().cuda_stream) == 0
    torch.cuda.synchronize()
    return lab.cpu().numpy()


def _cases():
    rng = np.random.default_rng(31)
    yield "ties", (rng.integers(0, 9, size=(37, 6)) / 8.0).astype(F)
    yield "js-like", (rng.gamma(0.7, 0.12, size=(300, 8)).clip(0, 0.6931)).astype(F)
    yield "one-row", rng.random((1, 20), dtype=F)
    yield "one-position", rng.random((50, 1), dtype=F)
    d = rng.random((64, 9), dtype=F)
    d[rng.random((64, 9)) < 0.05] = np.nan
    d[rng.random((64, 9)) < 0.05] = np.inf
    d[rng.random((64, 9)) < 0.1] = 0.0
    yield "nan-inf-zero", d
    yield "many-rows", rng.random((5000, 12), dtype=F)            # more rows than threads


@pytest.mark.parametrize("cmp", ["lt", "le"])
def test_sweep_calibrate_and_labels_match_the_oracle(cmp):
    for name, D in _cases():
        B, G = D.shape
        finite = D[np.isfinite(D)]
        Ts = np.concatenate([[0.0, 0.1, 0.2, 0.5, 0.6931, 1e9, np.inf], finite[:5],
                             np.nextafter(finite[:3], F(np.inf))]).astype(F)
        m, f = _gpu_sweep(D, Ts, cmp)
        om, of = tun.threshold_sweep(D, Ts, cmp)
        assert np.array_equal(m, om) and np.array_equal(f, of), name
        for T in (0.0, 0.3, float(finite[0])):
            assert np.array_equal(_gpu_labels(D, T, cmp), tun.accept_labels(D, T, cmp)), name
        if B * G <= 3000:                                         # the oracle's exhaustive search is quadratic
            for target in (0.0, 0.25, 1.0, G / 2, G - 0.5, float(G), G + 3.0):
                T, got = _gpu_calibrate(D, target, cmp)
                oT, ogot = tun.calibrate_threshold(D, target, cmp)
                assert (T == oT or (np.isinf(T) and np.isinf(oT))) and got == ogot, (name, target, T, oT, got, ogot)


def test_calibrated_threshold_reproduces_itself_through_the_sweep():
    """At full size (too large for the oracle's exhaustive search): the threshold found must reach
    the target in the sweep, and the next float below it must not."""
    rng = np.random.default_rng(32)
    D = rng.gamma(0.7, 0.12, size=(20000, 8)).clip(0, 0.6931).astype(F)
    for cmp in ("lt", "le"):
        for target in (0.5, 2.0, 5.5, 7.99):
            T, got = _gpu_calibrate(D, target, cmp)
            below = np.nextafter(F(T), F(-np.inf))
            m, _ = _gpu_sweep(D, [T, below], cmp)
            assert m[0] == got and m[0] >= F(target) and m[1] < F(target)
            # and the sweep itself is the definition on sampled rows
            idx = rng.choice(D.shape[0], 400, replace=False)
            sm, _ = _gpu_sweep(D[idx], [T], cmp)
            assert sm[0] == tun.threshold_sweep(D[idx], [T], cmp)[0][0]


def test_tuning_on_divergences_of_a_verify_call_reproduces_its_accept_lengths():
    import fsd_inputs as gi
    from tests import parity
    c = gi.make_chain(12, 6, 4096, dtype="bf16", recipe="spike", sigma=(0.2, 1.5), sigma_mode="uniform", workload_id=778)
    for T in (0.05, 0.3):
        g = parity.run_chain_gpu(c.target, c.draft, None, None, c.u_sample, c.dtype, T=T)
        D = g.divergence.astype(F)
        m, _ = _gpu_sweep(D, [T], "lt")
        assert m[0] == F(g.accept_len.sum() / 12)
        assert np.array_equal(_gpu_labels(D, T, "lt"), (D < F(T)).astype(np.uint8))
