"""ctypes front end of the CPU oracle (``fsd_oracle.c``).

TEST INFRASTRUCTURE.  Only tests, the smoke check and the benchmark's
CPU-baseline leg may import this module; the product never does.  The arithmetic
lives in the C file; this module only marshals numpy arrays.
"""

from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fsd_oracle.c")
_LIB = os.path.join(_HERE, "libfsd_oracle.so")

DTYPES = {"f32": 0, "bf16": 1}
DIVS = {"js": 0, "kl": 1, "tv": 2}
MODES = {"fsd": 0, "sd": 1, "rfsd": 2}
CMPS = {"lt": 0, "le": 1}
SAMPLES = {"invcdf": 0, "greedy": 1}

ST_NONFINITE = 1
ST_BADTREE = 4


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, OpenMP for the outer loops)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        l = C.CDLL(build())
        dp, ip, vp, fp, bp = (C.POINTER(C.c_double), C.POINTER(C.c_int32), C.c_void_p,
                              C.POINTER(C.c_float), C.POINTER(C.c_int8))
        l.fsd_oracle_softmax.argtypes = [vp, C.c_int, C.c_int, dp]
        l.fsd_oracle_softmax.restype = C.c_int
        l.fsd_oracle_divergence_probs.argtypes = [dp, dp, C.c_int, C.c_int]
        l.fsd_oracle_divergence_probs.restype = C.c_double
        l.fsd_oracle_divergence_logits.argtypes = [vp, vp, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int)]
        l.fsd_oracle_divergence_logits.restype = C.c_double
        l.fsd_oracle_sd_accept_prob.argtypes = [C.c_double, C.c_double]
        l.fsd_oracle_sd_accept_prob.restype = C.c_double
        l.fsd_oracle_sample.argtypes = [dp, C.c_int, C.c_double, C.c_double, C.POINTER(C.c_int),
                                        C.POINTER(C.c_int), dp]
        l.fsd_oracle_sample.restype = C.c_int
        l.fsd_oracle_argmax.argtypes = [dp, C.c_int]
        l.fsd_oracle_argmax.restype = C.c_int
        l.fsd_oracle_chain.argtypes = [vp, vp, ip, fp, fp] + [C.c_int] * 8 + [C.c_double, C.c_double, bp,
                                                                           ip, ip, dp, dp, bp, ip, ip, dp, ip, C.c_int]
        l.fsd_oracle_chain.restype = C.c_int
        l.fsd_oracle_tree.argtypes = [vp, vp, ip, fp] + [C.c_int] * 8 + [C.c_double, C.c_double, bp,
                                                                      ip, ip, ip, dp, bp, ip, ip, ip, dp, ip, C.c_int]
        l.fsd_oracle_tree.restype = C.c_int
        l.fsd_oracle_max_threads.restype = C.c_int
        _lib = l
    return _lib


def _p(a: Optional[np.ndarray], ctype):
    return None if a is None else a.ctypes.data_as(C.POINTER(ctype))


def _logits(a: np.ndarray, dtype: str) -> np.ndarray:
    want = np.uint16 if dtype == "bf16" else np.float32
    a = np.ascontiguousarray(a)
    if a.dtype != want:
        raise TypeError(f"{dtype} logits must be {want}, got {a.dtype}")
    return a


def softmax(logits: np.ndarray, dtype: str = "f32"):
    a = _logits(logits, dtype)
    p = np.empty(a.shape[-1], dtype=np.float64)
    st = lib().fsd_oracle_softmax(a.ctypes.data, a.shape[-1], DTYPES[dtype], _p(p, C.c_double))
    return p, st


def divergence_probs(p, q, kind: str = "js") -> float:
    p = np.ascontiguousarray(p, dtype=np.float64)
    q = np.ascontiguousarray(q, dtype=np.float64)
    return lib().fsd_oracle_divergence_probs(_p(p, C.c_double), _p(q, C.c_double), p.shape[0], DIVS[kind])


def divergence_logits(a, b, kind: str = "js", dtype: str = "f32") -> float:
    a = _logits(a, dtype)
    b = _logits(b, dtype)
    st = C.c_int(0)
    return lib().fsd_oracle_divergence_logits(a.ctypes.data, b.ctypes.data, a.shape[-1], DTYPES[dtype],
                                              DIVS[kind], C.byref(st))


def sd_accept_prob(p_x: float, q_x: float) -> float:
    return lib().fsd_oracle_sd_accept_prob(p_x, q_x)


def sample(w, u: float, band: float = 0.0):
    """Returns (token, tok_lo, tok_hi, margin)."""
    w = np.ascontiguousarray(w, dtype=np.float64)
    lo, hi, mg = C.c_int(0), C.c_int(0), C.c_double(0.0)
    tok = lib().fsd_oracle_sample(_p(w, C.c_double), w.shape[0], u, band, C.byref(lo), C.byref(hi), C.byref(mg))
    return tok, lo.value, hi.value, mg.value


def argmax(w) -> int:
    w = np.ascontiguousarray(w, dtype=np.float64)
    return lib().fsd_oracle_argmax(_p(w, C.c_double), w.shape[0])


@dataclass
class ChainResult:
    accept_len: np.ndarray      # [B] int32
    next_token: np.ndarray      # [B] int32
    divergence: np.ndarray      # [B, gamma] float64
    p_accept: np.ndarray        # [B, gamma] float64 (NaN where no draft token was given)
    accept_bits: np.ndarray     # [B, gamma] int8
    tok_lo: np.ndarray          # [B] int32
    tok_hi: np.ndarray          # [B] int32
    margin: np.ndarray          # [B] float64
    row_status: np.ndarray      # [B] int32


def verify_chain(target, draft, draft_tokens, u_accept, u_sample, dtype="bf16", div="js", mode="fsd",
                 cmp="lt", sample_kind="invcdf", T=0.2, band=0.0, forced=None, nthreads=0) -> ChainResult:
    target = _logits(target, dtype)
    draft = _logits(draft, dtype)
    B, g1, V = target.shape
    gamma = g1 - 1
    assert draft.shape == (B, gamma, V)
    tok = None if draft_tokens is None else np.ascontiguousarray(draft_tokens, dtype=np.int32)
    ua = None if u_accept is None else np.ascontiguousarray(u_accept, dtype=np.float32)
    us = np.ascontiguousarray(u_sample, dtype=np.float32)
    fo = None if forced is None else np.ascontiguousarray(forced, dtype=np.int8)
    r = ChainResult(np.empty(B, np.int32), np.empty(B, np.int32), np.empty((B, gamma)), np.empty((B, gamma)),
                    np.empty((B, gamma), np.int8), np.empty(B, np.int32), np.empty(B, np.int32), np.empty(B),
                    np.empty(B, np.int32))
    rc = lib().fsd_oracle_chain(target.ctypes.data, draft.ctypes.data, _p(tok, C.c_int32), _p(ua, C.c_float),
                                _p(us, C.c_float), B, gamma, V, DTYPES[dtype], DIVS[div], MODES[mode], CMPS[cmp],
                                SAMPLES[sample_kind], float(T), float(band), _p(fo, C.c_int8),
                                _p(r.accept_len, C.c_int32), _p(r.next_token, C.c_int32),
                                _p(r.divergence, C.c_double), _p(r.p_accept, C.c_double),
                                _p(r.accept_bits, C.c_int8), _p(r.tok_lo, C.c_int32), _p(r.tok_hi, C.c_int32),
                                _p(r.margin, C.c_double), _p(r.row_status, C.c_int32), int(nthreads))
    if rc != 0:
        raise ValueError(f"fsd_oracle_chain failed with {rc}")
    return r


@dataclass
class TreeResult:
    accept_len: np.ndarray      # [B] depth of the chosen node
    path: np.ndarray            # [B, max_depth] node ids, -1 padded
    next_token: np.ndarray
    divergence: np.ndarray      # [B, N]
    accept_bits: np.ndarray     # [B, N] per-node test (before ancestors are considered)
    end_node: np.ndarray        # [B] chosen node id, -1 = root
    tok_lo: np.ndarray
    tok_hi: np.ndarray
    margin: np.ndarray
    row_status: np.ndarray


def verify_tree(target, draft, parent, u_sample, max_depth, dtype="bf16", div="js", cmp="lt",
                sample_kind="invcdf", T=0.2, band=0.0, forced=None, nthreads=0) -> TreeResult:
    target = _logits(target, dtype)
    draft = _logits(draft, dtype)
    B, n1, V = target.shape
    N = n1 - 1
    assert draft.shape == (B, N, V)
    par = np.ascontiguousarray(parent, dtype=np.int32)
    assert par.shape == (B, N)
    us = np.ascontiguousarray(u_sample, dtype=np.float32)
    fo = None if forced is None else np.ascontiguousarray(forced, dtype=np.int8)
    r = TreeResult(np.empty(B, np.int32), np.empty((B, max_depth), np.int32), np.empty(B, np.int32),
                   np.empty((B, N)), np.empty((B, N), np.int8), np.empty(B, np.int32), np.empty(B, np.int32),
                   np.empty(B, np.int32), np.empty(B), np.empty(B, np.int32))
    rc = lib().fsd_oracle_tree(target.ctypes.data, draft.ctypes.data, _p(par, C.c_int32), _p(us, C.c_float),
                               B, N, V, int(max_depth), DTYPES[dtype], DIVS[div], CMPS[cmp], SAMPLES[sample_kind],
                               float(T), float(band), _p(fo, C.c_int8),
                               _p(r.accept_len, C.c_int32), _p(r.path, C.c_int32), _p(r.next_token, C.c_int32),
                               _p(r.divergence, C.c_double), _p(r.accept_bits, C.c_int8), _p(r.end_node, C.c_int32),
                               _p(r.tok_lo, C.c_int32), _p(r.tok_hi, C.c_int32), _p(r.margin, C.c_double),
                               _p(r.row_status, C.c_int32), int(nthreads))
    if rc != 0:
        raise ValueError(f"fsd_oracle_tree failed with {rc}")
    return r


def max_threads() -> int:
    return lib().fsd_oracle_max_threads()
