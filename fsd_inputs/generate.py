"""Seeded generators for chain and tree verification inputs.

Everything is produced on the host with numpy's counter-based Philox bit
generator, keyed by (base seed, workload id, tensor id, batch row, position),
so any single row can be regenerated on its own and a workload is the same on
every machine that runs the same numpy.

Two logit recipes are used:

* ``spike``: ``a = 3 * N(0, 1)`` with ``+8`` added at one seeded index.  Gives a
  moderately peaked distribution (largest probability around 0.1).
* ``zipf``: ``a_k = -1.1 * ln(rank_k) + N(0, 0.5)`` where ``rank`` is a seeded
  permutation of ``1..V``.  Gives the heavy-tailed shape of a language model's
  next-token distribution.

Draft rows are the (unrounded) target row plus ``N(0, sigma)`` noise; a
``disjoint`` draft row is instead a fresh ``zipf`` row under an independent
permutation, which makes the two distributions nearly disjoint.

Draft tokens are drawn from the categorical distribution whose logits are the
draft row by the Gumbel-max construction (argmax of logits plus Gumbel noise),
which needs no normalisation.

bf16 tensors are returned as ``uint16`` bit patterns (round-to-nearest-even of
the float32 value); ``bf16_bits_to_f32`` widens them back exactly.
"""

from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional, Sequence

import numpy as np

BASE_SEED = 0x5EED250220704

# tensor ids used in the Philox key derivation
_T_TARGET, _T_DRAFT, _T_TOKENS, _T_UACC, _T_USAMP, _T_SIGMA, _T_DISJ, _T_TREE = range(8)


# --------------------------------------------------------------------------- #
# bf16 helpers (bit manipulation only)
# --------------------------------------------------------------------------- #
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to bfloat16 (nearest, ties to even); returns uint16 bits.

    ``-inf``/``+inf`` are preserved; NaN stays NaN (quiet bit forced).
    """
    x = np.ascontiguousarray(x, dtype=np.float32)
    bits = x.view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    rounded = (bits + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    out = rounded.astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = ((bits[nan] >> np.uint32(16)) | np.uint32(0x0040)).astype(np.uint16)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to float32 exactly."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(*key: int) -> np.random.Generator:
    ss = np.random.SeedSequence([BASE_SEED & 0xFFFFFFFF, BASE_SEED >> 32, *[int(k) & 0xFFFFFFFF for k in key]])
    return np.random.Generator(np.random.Philox(ss))


# --------------------------------------------------------------------------- #
# row recipes (float32, before rounding to the storage dtype)
# --------------------------------------------------------------------------- #
def _spike_row(rng: np.random.Generator, V: int) -> np.ndarray:
    a = rng.standard_normal(V, dtype=np.float32) * np.float32(3.0)
    k = int(rng.integers(0, V))
    a[k] += np.float32(8.0)
    return a


def _zipf_row(rng: np.random.Generator, V: int) -> np.ndarray:
    rank = rng.permutation(V).astype(np.float32) + np.float32(1.0)
    noise = rng.standard_normal(V, dtype=np.float32) * np.float32(0.5)
    return np.float32(-1.1) * np.log(rank) + noise


_RECIPES = {"spike": _spike_row, "zipf": _zipf_row}


def _gumbel_argmax(rng: np.random.Generator, logits_f32: np.ndarray) -> int:
    u = rng.random(logits_f32.shape[0])
    with np.errstate(divide="ignore"):
        g = -np.log(-np.log(u))
    return int(np.argmax(logits_f32.astype(np.float64) + g))


def _store(row_f32: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return f32_to_bf16_bits(row_f32)
    return row_f32.astype(np.float32)


def _stored_as_f32(stored: np.ndarray, dtype: str) -> np.ndarray:
    return bf16_bits_to_f32(stored) if dtype == "bf16" else stored


# --------------------------------------------------------------------------- #
# containers
# --------------------------------------------------------------------------- #
@dataclass
class ChainInputs:
    B: int
    gamma: int
    V: int
    dtype: str                      # "f32" | "bf16"
    target: np.ndarray              # [B, gamma+1, V]  float32 or uint16 (bf16 bits)
    draft: np.ndarray               # [B, gamma,   V]
    draft_tokens: np.ndarray        # [B, gamma] int32
    u_accept: np.ndarray            # [B, gamma] float32 in [0,1)
    u_sample: np.ndarray            # [B] float32 in [0,1)
    sigma: np.ndarray               # [B, gamma] float64 noise scale used per position
    disjoint: np.ndarray            # [B, gamma] bool

    @property
    def elem_size(self) -> int:
        return 2 if self.dtype == "bf16" else 4

    @property
    def ideal_bytes(self) -> int:
        """Each logit the result depends on, read once: (2*gamma+1) rows per batch row."""
        return self.elem_size * self.B * (2 * self.gamma + 1) * self.V


@dataclass
class TreeInputs:
    B: int
    N: int
    V: int
    dtype: str
    max_depth: int
    target: np.ndarray              # [B, N+1, V]; row 0 = root context, row j+1 = context ending in node j
    draft: np.ndarray               # [B, N,   V]; row j = distribution node j was proposed from
    parent: np.ndarray              # [B, N] int32; -1 = child of the root; parent[j] < j
    draft_tokens: np.ndarray        # [B, N] int32
    u_sample: np.ndarray            # [B] float32

    @property
    def elem_size(self) -> int:
        return 2 if self.dtype == "bf16" else 4


# --------------------------------------------------------------------------- #
# chain workloads
# --------------------------------------------------------------------------- #
def make_chain(
    B: int,
    gamma: int,
    V: int,
    dtype: str = "bf16",
    recipe: str = "spike",
    sigma: Sequence[float] | tuple = (0.1, 0.5, 2.0),
    sigma_mode: str = "cycle",          # "cycle": sigma[i % len]; "uniform": U(sigma[0], sigma[1]) per (b, i)
    disjoint_frac: float = 0.0,
    workload_id: int = 0,
) -> ChainInputs:
    if dtype not in ("f32", "bf16"):
        raise ValueError("dtype must be 'f32' or 'bf16'")
    row_fn = _RECIPES[recipe]
    np_dt = np.uint16 if dtype == "bf16" else np.float32
    target = np.empty((B, gamma + 1, V), dtype=np_dt)
    draft = np.empty((B, gamma, V), dtype=np_dt)
    tokens = np.empty((B, gamma), dtype=np.int32)
    sig = np.empty((B, gamma), dtype=np.float64)
    disj = np.zeros((B, gamma), dtype=bool)

    for b in range(B):
        for i in range(gamma + 1):
            a = row_fn(_rng(workload_id, _T_TARGET, b, i), V)
            target[b, i] = _store(a, dtype)
            if i == gamma:
                break
            r = _rng(workload_id, _T_SIGMA, b, i)
            if sigma_mode == "cycle":
                s = float(sigma[i % len(sigma)])
            else:
                s = float(r.uniform(sigma[0], sigma[1]))
            sig[b, i] = s
            is_disj = bool(_rng(workload_id, _T_DISJ, b, i).random() < disjoint_frac)
            disj[b, i] = is_disj
            rd = _rng(workload_id, _T_DRAFT, b, i)
            if is_disj:
                d = _zipf_row(rd, V)
            else:
                d = a + rd.standard_normal(V, dtype=np.float32) * np.float32(s)
            draft[b, i] = _store(d, dtype)
            tokens[b, i] = _gumbel_argmax(_rng(workload_id, _T_TOKENS, b, i), _stored_as_f32(draft[b, i], dtype))

    u_acc = _rng(workload_id, _T_UACC).random((B, gamma), dtype=np.float32)
    u_smp = _rng(workload_id, _T_USAMP).random(B, dtype=np.float32)
    return ChainInputs(B, gamma, V, dtype, target, draft, tokens, u_acc, u_smp, sig, disj)


# --------------------------------------------------------------------------- #
# tree workloads
# --------------------------------------------------------------------------- #
def _random_parents(rng: np.random.Generator, N: int, max_depth: int, max_children: int) -> np.ndarray:
    """Seeded draft tree: parent[j] in [-1, j), depth <= max_depth, at most max_children per node."""
    parent = np.empty(N, dtype=np.int32)
    depth = np.zeros(N, dtype=np.int32)
    nchild = np.zeros(N + 1, dtype=np.int32)  # slot 0 = root, slot j+1 = node j
    for j in range(N):
        elig = [-1] if nchild[0] < max_children else []
        elig += [i for i in range(j) if nchild[i + 1] < max_children and depth[i] < max_depth]
        if not elig:
            raise ValueError("tree cannot hold N nodes under the depth/branching limits")
        p = int(elig[int(rng.integers(0, len(elig)))])
        parent[j] = p
        depth[j] = 1 if p < 0 else depth[p] + 1
        nchild[p + 1] += 1
    return parent


def make_tree(
    B: int,
    N: int,
    V: int,
    dtype: str = "bf16",
    recipe: str = "spike",
    sigma: float = 0.6,
    max_depth: int = 6,
    max_children: int = 4,
    workload_id: int = 0,
    parent: Optional[np.ndarray] = None,
) -> TreeInputs:
    row_fn = _RECIPES[recipe]
    np_dt = np.uint16 if dtype == "bf16" else np.float32
    target = np.empty((B, N + 1, V), dtype=np_dt)
    draft = np.empty((B, N, V), dtype=np_dt)
    tokens = np.empty((B, N), dtype=np.int32)
    if parent is None:
        par = np.stack([_random_parents(_rng(workload_id, _T_TREE, b), N, max_depth, max_children) for b in range(B)])
    else:
        par = np.broadcast_to(np.asarray(parent, dtype=np.int32), (B, N)).copy()
    for b in range(B):
        rows_f32 = []
        for r in range(N + 1):
            a = row_fn(_rng(workload_id, _T_TARGET, b, r), V)
            rows_f32.append(a)
            target[b, r] = _store(a, dtype)
        for j in range(N):
            base = rows_f32[int(par[b, j]) + 1]
            rd = _rng(workload_id, _T_DRAFT, b, j)
            d = base + rd.standard_normal(V, dtype=np.float32) * np.float32(sigma)
            draft[b, j] = _store(d, dtype)
            tokens[b, j] = _gumbel_argmax(_rng(workload_id, _T_TOKENS, b, j), _stored_as_f32(draft[b, j], dtype))
    u_smp = _rng(workload_id, _T_USAMP).random(B, dtype=np.float32)
    return TreeInputs(B, N, V, dtype, max_depth, target, draft, par, tokens, u_smp)


def tree_unique_rows(parent: np.ndarray, end_node: np.ndarray) -> int:
    """Number of distinct logit rows a tree verification depends on.

    Per batch row: the N draft rows, every target row that is some node's parent
    context (row 0 for children of the root), and the target row after the chosen
    end node (``end_node[b]`` = node id, or -1 for the root) when it is not already
    among those.
    """
    parent = np.asarray(parent)
    total = 0
    for b in range(parent.shape[0]):
        rows = set(int(p) + 1 for p in parent[b])
        rows.add(int(end_node[b]) + 1)
        total += parent.shape[1] + len(rows)
    return total


# --------------------------------------------------------------------------- #
# the five named workloads
# --------------------------------------------------------------------------- #
@dataclass
class ConfigSpec:
    name: str
    kind: str                       # "chain" | "tree"
    params: Dict = field(default_factory=dict)
    thresholds: Sequence[float] = ()
    modes: Sequence[str] = ("fsd",)
    divergences: Sequence[str] = ("js",)


CONFIGS: Dict[str, ConfigSpec] = {
    "c1": ConfigSpec(
        "c1", "chain",
        dict(B=1, gamma=4, V=32000, dtype="f32", recipe="spike", sigma=(0.1, 0.5, 2.0), sigma_mode="cycle", workload_id=1),
        thresholds=(0.0, 0.05, 0.2, 1.0), divergences=("js", "kl", "tv")),
    "c2": ConfigSpec(
        "c2", "chain",
        dict(B=16, gamma=5, V=32000, dtype="bf16", recipe="spike", sigma=(0.1, 1.5), sigma_mode="uniform", workload_id=2),
        thresholds=tuple(k / 7.0 for k in range(8)), modes=("fsd", "sd")),
    "c3": ConfigSpec(
        "c3", "chain",
        dict(B=32, gamma=6, V=128256, dtype="bf16", recipe="zipf", sigma=(0.8,), sigma_mode="cycle", disjoint_frac=0.10, workload_id=3),
        thresholds=(0.1, 0.3)),
    "c4": ConfigSpec(
        "c4", "chain",
        dict(B=64, gamma=8, V=152064, dtype="bf16", recipe="zipf", sigma=(0.2, 2.0), sigma_mode="uniform", disjoint_frac=0.10, workload_id=4),
        thresholds=(0.2,)),
    "c5": ConfigSpec(
        "c5", "tree",
        dict(B=8, N=60, V=32000, dtype="bf16", recipe="spike", sigma=0.6, max_depth=6, max_children=4, workload_id=5),
        thresholds=(0.05, 0.2, 0.5)),
}


def make_config(name: str, **overrides):
    """Build one of the named workloads; ``overrides`` replace generator parameters (e.g. a smaller B)."""
    spec = CONFIGS[name]
    params = dict(spec.params)
    params.update(overrides)
    return make_chain(**params) if spec.kind == "chain" else make_tree(**params)
