"""Pins of the threshold-tuning oracle (oracle/fsd_tuning_oracle.py): worked cases, closed forms,
agreement with the pinned verification oracle, minimality by exhaustive search."""

import numpy as np
import pytest

import fsd_inputs as gi
from oracle import fsd_oracle as orc
from oracle import fsd_tuning_oracle as tun

F = np.float32


def test_worked_case_by_hand():
    D = np.array([[0.1, 0.5, 0.2], [0.3, 0.05, 0.9]], dtype=F)
    # T = 0.25: row 0 stops at 0.5 (1 accepted), row 1 stops at once (0)
    assert tun.accepted_lengths(D, 0.25).tolist() == [1, 0]
    # T = 0.6: row 0 passes everything (3), row 1 stops at 0.9 (2)
    assert tun.accepted_lengths(D, 0.6).tolist() == [3, 2]
    mean, frac = tun.threshold_sweep(D, [0.25, 0.6, 1.0])
    assert mean.tolist() == [0.5, 2.5, 3.0]
    assert np.allclose(frac, [1 / 6, 5 / 6, 1.0], rtol=0, atol=1e-7)
    # labels look at each position alone: 0.2 and 0.05 pass at T = 0.25 although their prefixes failed
    assert tun.accept_labels(D, 0.25).tolist() == [[1, 0, 1], [0, 1, 0]]
    # mean length 1.0 needs 2 accepted positions.  Up to T = 0.3 only (0,0) = 0.1 passes (1 position);
    # once 0.3 passes, row 1 takes 0.3 and the 0.05 behind it: 3 positions, mean 1.5.  So T must
    # exceed 0.3 under < and equal it under <=
    T, got = tun.calibrate_threshold(D, 1.0, "lt")
    assert T == np.nextafter(F(0.3), F(np.inf)) and got == 1.5
    T, got = tun.calibrate_threshold(D, 1.0, "le")
    assert T == F(0.3) and got == 1.5
    # 2.5 needs 5: everything but the 0.9
    T, got = tun.calibrate_threshold(D, 2.5, "le")
    assert T == F(0.5) and got == 2.5


def test_strict_and_nonstrict_differ_only_at_equality():
    D = np.array([[0.25, 0.25, 0.5]], dtype=F)
    assert tun.accepted_lengths(D, 0.25, "lt").tolist() == [0]
    assert tun.accepted_lengths(D, 0.25, "le").tolist() == [2]
    assert tun.accepted_lengths(D, 0.26, "lt").tolist() == tun.accepted_lengths(D, 0.26, "le").tolist() == [2]
    # T = 0 under < accepts nothing, under <= exactly the zero divergences (identical rows)
    Z = np.array([[0.0, 0.0, 0.1], [0.0, 0.2, 0.0]], dtype=F)
    assert tun.accepted_lengths(Z, 0.0, "lt").tolist() == [0, 0]
    assert tun.accepted_lengths(Z, 0.0, "le").tolist() == [2, 1]


def test_nan_and_infinite_divergences():
    D = np.array([[0.1, np.nan, 0.1], [0.1, np.inf, 0.1]], dtype=F)
    assert tun.accepted_lengths(D, 10.0).tolist() == [1, 1]
    assert tun.accepted_lengths(D, np.inf, "lt").tolist() == [1, 1]
    assert tun.accepted_lengths(D, np.inf, "le").tolist() == [1, 3]          # inf <= inf
    assert tun.accept_labels(D, 1.0).tolist() == [[1, 0, 1], [1, 0, 1]]
    # a target nobody can reach with a finite threshold
    T, got = tun.calibrate_threshold(D, 2.0, "lt")
    assert np.isposinf(T) and got == 1.0


def test_monotone_and_extremes():
    rng = np.random.default_rng(1)
    D = rng.random((7, 9), dtype=F)
    prev = -1.0
    for T in np.linspace(0.0, 1.1, 23):
        n = tun.accepted_lengths(D, T)
        assert n.sum() >= prev
        prev = n.sum()
    assert tun.accepted_lengths(D, 0.0).sum() == 0
    assert tun.accepted_lengths(D, 2.0).tolist() == [9] * 7
    mean, frac = tun.threshold_sweep(D, [2.0])
    assert mean[0] == 9.0 and frac[0] == 1.0


def test_constant_divergence_closed_form():
    D = np.full((5, 4), 0.37, dtype=F)
    for target in (0.5, 3.9, 4.0):
        T, got = tun.calibrate_threshold(D, target, "lt")
        assert T == np.nextafter(F(0.37), F(np.inf)) and got == 4.0            # all or nothing
        T, got = tun.calibrate_threshold(D, target, "le")
        assert T == F(0.37) and got == 4.0
    T, got = tun.calibrate_threshold(D, 0.0, "lt")
    assert T == 0.0 and got == 0.0


@pytest.mark.parametrize("cmp", ["lt", "le"])
def test_calibrated_threshold_is_minimal(cmp):
    rng = np.random.default_rng(2)
    for trial in range(40):
        B, G = int(rng.integers(1, 6)), int(rng.integers(1, 6))
        D = (rng.integers(0, 6, size=(B, G)) / 8.0).astype(F)                # many ties
        target = float(rng.integers(0, 4 * G + 1)) / 4.0
        T, got = tun.calibrate_threshold(D, target, cmp)
        need = min(max(int(np.ceil(target * B)), 0), B * G)
        assert int(tun.accepted_lengths(D, T, cmp).sum()) >= need
        assert got == F(tun.accepted_lengths(D, T, cmp).sum() / B)
        if T > 0:                                                           # the next float down falls short
            below = np.nextafter(T, F(-np.inf))
            assert int(tun.accepted_lengths(D, below, cmp).sum()) < need


def test_agrees_with_the_verification_oracle_on_real_divergences():
    c = gi.make_chain(6, 5, 512, dtype="f32", recipe="spike", sigma=(0.2, 1.5), sigma_mode="uniform", workload_id=777)
    for cmp in ("lt", "le"):
        for T in (0.0, 0.05, 0.2, 0.6):
            r = orc.verify_chain(c.target, c.draft, None, None, c.u_sample, dtype="f32", div="js", mode="fsd",
                                 cmp=cmp, T=T)
            D32 = r.divergence.astype(F)
            # the verification oracle decides in double; stay away from float32 rounding of D at T
            if np.any(np.abs(r.divergence - float(F(T))) < 1e-6):
                continue
            assert tun.accepted_lengths(D32, T, cmp).tolist() == r.accept_len.tolist()
