"""Helpers for the GPU-vs-oracle parity tests: run the CUDA library through its C ABI on
seeded inputs, run the CPU oracle on the same inputs, and compare under the stated rules.

Rules
  * divergences agree within `tol` absolute (1e-5 for fp32 logits, 1e-4 for bf16); infinities
    and NaNs must coincide.
  * a batch row is "band-affected" when some position up to the later of the two accepted
    lengths has |D_oracle - T| < 1e-5 (FSD, rFSD) or |P_accept - u| < 1e-6 (SD, rFSD): there the
    fp32 and fp64 decisions may legitimately differ.  Unaffected rows must match bit-exactly in
    accept_len and next_token.  Affected rows are replayed: the oracle is re-run with the in-band
    decisions forced to what the GPU's accept_len implies and must then reproduce the GPU's
    accept_len and token.
  * tokens: the oracle reports the tokens selected for t -/+ band*W; a GPU token inside that
    range but different from the oracle's is counted as a sample-band hit, one outside fails.
    A token drawn from P_T (every FSD draw, every bonus token) is computed on the GPU from
    single-precision exponentials summed in double: band = 1e-6, so the token is the oracle's
    own whenever u*W is further than 1e-6*W from both ends of that token's interval.  A token
    drawn from the SD residual max(0, P_T - P_D) is computed in double throughout and differs
    from the sequential sum by rounding only: band = 1e-12.
"""

from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

import paper_2502_20704_b200 as fsd
from oracle import fsd_oracle as orc

D_BAND = 1e-5
P_BAND = 1e-6
SAMPLE_BAND_PT = 1e-6          # draws from P_T
SAMPLE_BAND_RESIDUAL = 1e-12   # draws from the SD residual
SAMPLE_BAND = SAMPLE_BAND_PT   # tree verification and FSD mode draw from P_T only


def to_device(arr: np.ndarray, dtype: str):
    if arr is None:
        return None
    if arr.dtype == np.uint16:
        return torch.from_numpy(arr.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(arr).cuda()


@dataclass
class GpuChain:
    accept_len: np.ndarray
    next_token: np.ndarray
    divergence: np.ndarray
    row_status: np.ndarray


def run_chain_gpu(target, draft, tokens, u_accept, u_sample, dtype, div="js", mode="fsd", cmp="lt",
                  sample="invcdf", T=0.2, dev=None) -> GpuChain:
    B, g1, V = target.shape
    gamma = g1 - 1
    opts = fsd.make_opts(div=div, mode=mode, cmp=cmp, sample=sample, dtype=dtype, T=T)
    if dev is None:
        dev = dict(t=to_device(target, dtype), d=to_device(draft, dtype), tok=to_device(tokens, dtype),
                   ua=to_device(u_accept, dtype), us=to_device(u_sample, dtype))
    acc = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    tok = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    D = torch.full((B, gamma), -7.0, dtype=torch.float32, device="cuda")
    st = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    wsb = fsd.fsd_workspace_bytes(B, gamma, V, opts)
    ws = torch.empty(wsb + 256, dtype=torch.uint8, device="cuda")
    ws.fill_(0xAB)                      # the library must not rely on zeroed scratch
    rc = fsd.fsd_verify_chain(dev["t"], dev["d"], dev["tok"], dev["ua"], dev["us"], B, gamma, V, opts,
                              acc, tok, D, st, ws, wsb, torch.cuda.current_stream().cuda_stream)
    assert rc == 0, fsd.fsd_status_string(rc)
    torch.cuda.synchronize()
    assert (ws[wsb:] == 0xAB).all(), "workspace overrun"
    return GpuChain(acc.cpu().numpy(), tok.cpu().numpy(), D.cpu().numpy(), st.cpu().numpy())


@dataclass
class GpuTree:
    accept_len: np.ndarray
    path: np.ndarray
    next_token: np.ndarray
    divergence: np.ndarray
    row_status: np.ndarray


def run_tree_gpu(target, draft, parent, u_sample, max_depth, dtype, div="js", cmp="lt", sample="invcdf",
                 T=0.2) -> GpuTree:
    B, n1, V = target.shape
    N = n1 - 1
    opts = fsd.make_opts(div=div, mode="fsd", cmp=cmp, sample=sample, dtype=dtype, T=T)
    t, d = to_device(target, dtype), to_device(draft, dtype)
    par, us = to_device(np.ascontiguousarray(parent, np.int32), dtype), to_device(u_sample, dtype)
    acc = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    path = torch.full((B, max_depth), -7, dtype=torch.int32, device="cuda")
    tok = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    D = torch.full((B, N), -7.0, dtype=torch.float32, device="cuda")
    st = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    wsb = fsd.fsd_workspace_bytes(B, N, V, opts)
    ws = torch.empty(wsb + 256, dtype=torch.uint8, device="cuda")
    ws.fill_(0xAB)
    rc = fsd.fsd_verify_tree(t, d, par, us, B, N, V, max_depth, opts, acc, path, tok, D, st, ws, wsb,
                             torch.cuda.current_stream().cuda_stream)
    assert rc == 0, fsd.fsd_status_string(rc)
    torch.cuda.synchronize()
    assert (ws[wsb:] == 0xAB).all(), "workspace overrun"
    return GpuTree(acc.cpu().numpy(), path.cpu().numpy(), tok.cpu().numpy(), D.cpu().numpy(), st.cpu().numpy())


def compare_divergence(D_gpu, D_orc, tol):
    D_gpu = np.asarray(D_gpu, dtype=np.float64)
    fin = np.isfinite(D_orc)
    assert np.array_equal(np.isnan(D_gpu), np.isnan(D_orc)), "NaN pattern differs"
    assert np.array_equal(np.isposinf(D_gpu), np.isposinf(D_orc)), "inf pattern differs"
    err = np.abs(D_gpu[fin] - D_orc[fin])
    mx = float(err.max()) if err.size else 0.0
    assert mx <= tol, f"divergence error {mx:.3e} > {tol:.1e}"
    return mx


def check_chain(inp_target, inp_draft, tokens, u_accept, u_sample, dtype, div="js", mode="fsd", cmp="lt",
                sample="invcdf", T=0.2, dev=None):
    """Runs both sides and applies the parity rules; returns a dict of counts."""
    tol = 1e-5 if dtype == "f32" else 1e-4
    g = run_chain_gpu(inp_target, inp_draft, tokens, u_accept, u_sample, dtype, div, mode, cmp, sample, T, dev)
    o = orc.verify_chain(inp_target, inp_draft, tokens, u_accept, u_sample, dtype=dtype, div=div, mode=mode,
                         cmp=cmp, sample_kind=sample, T=T, band=SAMPLE_BAND_PT)
    B, gamma = o.divergence.shape
    # in SD / rFSD mode a rejected row draws from the residual: the tight band applies there
    o_res = None
    if mode != "fsd":
        o_res = orc.verify_chain(inp_target, inp_draft, tokens, u_accept, u_sample, dtype=dtype, div=div, mode=mode,
                                 cmp=cmp, sample_kind=sample, T=T, band=SAMPLE_BAND_RESIDUAL)

    def band_of(n_acc):
        return SAMPLE_BAND_RESIDUAL if (mode != "fsd" and n_acc < gamma) else SAMPLE_BAND_PT

    max_err = compare_divergence(g.divergence, o.divergence, tol)
    assert np.array_equal(g.row_status, o.row_status), (g.row_status, o.row_status)

    with np.errstate(invalid="ignore"):
        in_band = np.zeros((B, gamma), dtype=bool)
        if mode in ("fsd", "rfsd"):
            in_band |= np.abs(o.divergence - float(np.float32(T))) < D_BAND
        if mode in ("sd", "rfsd"):
            in_band |= np.abs(o.p_accept - u_accept.astype(np.float64)) < P_BAND
    band_rows, sample_band, replayed = 0, 0, 0
    for b in range(B):
        upto = min(gamma, max(int(g.accept_len[b]), int(o.accept_len[b])) + 1)
        affected = bool(in_band[b, :upto].any())
        n_o, t_o = int(o.accept_len[b]), int(o.next_token[b])
        src = o_res if (o_res is not None and n_o < gamma) else o
        lo, hi = int(src.tok_lo[b]), int(src.tok_hi[b])
        if affected and (g.accept_len[b] != n_o):
            band_rows += 1
            replayed += 1
            forced = np.full((1, gamma), -1, dtype=np.int8)
            for i in range(upto):
                if in_band[b, i]:
                    forced[0, i] = 1 if i < g.accept_len[b] else 0
            r = orc.verify_chain(inp_target[b:b + 1], inp_draft[b:b + 1],
                                 None if tokens is None else tokens[b:b + 1],
                                 None if u_accept is None else u_accept[b:b + 1], u_sample[b:b + 1],
                                 dtype=dtype, div=div, mode=mode, cmp=cmp, sample_kind=sample, T=T,
                                 band=band_of(int(g.accept_len[b])), forced=forced)
            n_o, t_o, lo, hi = int(r.accept_len[0]), int(r.next_token[0]), int(r.tok_lo[0]), int(r.tok_hi[0])
        elif affected:
            band_rows += 1
        assert g.accept_len[b] == n_o, f"row {b}: accept_len gpu {g.accept_len[b]} oracle {n_o}"
        if g.next_token[b] != t_o:
            assert lo <= g.next_token[b] <= hi, f"row {b}: token gpu {g.next_token[b]} oracle {t_o} [{lo},{hi}]"
            sample_band += 1
    return dict(rows=B, band_rows=band_rows, replayed=replayed, sample_band=sample_band, max_err=max_err,
                accept_len=g.accept_len.copy(), gpu=g, oracle=o)


def check_tree(c, T, div="js", cmp="lt", sample="invcdf"):
    """GPU tree verification against the oracle: divergences within tolerance; accepted depth, path
    and token identical, with the oracle re-run on the GPU's decisions where a divergence lies
    within D_BAND of the threshold."""
    tol = 1e-5 if c.dtype == "f32" else 1e-4
    g = run_tree_gpu(c.target, c.draft, c.parent, c.u_sample, c.max_depth, c.dtype, div=div, cmp=cmp, sample=sample, T=T)
    o = orc.verify_tree(c.target, c.draft, c.parent, c.u_sample, c.max_depth, dtype=c.dtype, div=div, cmp=cmp,
                        sample_kind=sample, T=T, band=SAMPLE_BAND)
    compare_divergence(g.divergence, o.divergence, tol)
    Tf = np.float32(T)
    with np.errstate(invalid="ignore"):
        in_band = np.abs(o.divergence - float(Tf)) < D_BAND
    for b in range(c.B):
        if in_band[b].any():
            forced = np.full((1, c.N), -1, dtype=np.int8)
            gd = g.divergence[b, in_band[b]]
            forced[0, in_band[b]] = ((gd <= Tf) if cmp == "le" else (gd < Tf)).astype(np.int8)
            ob = orc.verify_tree(c.target[b:b + 1], c.draft[b:b + 1], c.parent[b:b + 1], c.u_sample[b:b + 1],
                                 c.max_depth, dtype=c.dtype, div=div, cmp=cmp, sample_kind=sample, T=T,
                                 band=SAMPLE_BAND, forced=forced)
            n_o, p_o, t_o, lo, hi = ob.accept_len[0], ob.path[0], ob.next_token[0], ob.tok_lo[0], ob.tok_hi[0]
        else:
            n_o, p_o, t_o, lo, hi = o.accept_len[b], o.path[b], o.next_token[b], o.tok_lo[b], o.tok_hi[b]
        assert g.accept_len[b] == n_o and np.array_equal(g.path[b], p_o), f"row {b}"
        assert g.next_token[b] == t_o or lo <= g.next_token[b] <= hi, f"row {b}: token {g.next_token[b]} vs {t_o}"
    assert np.array_equal(g.row_status, o.row_status)
    return g, o
