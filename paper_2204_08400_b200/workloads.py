"""Seeded synthetic workloads (numpy only).

This module only draws random numbers and packs them; it holds none of the
method's arithmetic, so both the CUDA library's callers and the CPU checker's
callers may use it.  The shapes follow the paper's Table 1 architectures
(112-112 for the 784-feature image task, one 128-wide hidden layer in front of
a very wide output layer for the extreme-classification tasks) and the larger
MLPs named by this repository's benchmark configurations.  The paper's own
datasets and trained weights are not available; these draws stand in for them.
"""
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np


# ---- number-format helpers (storage format only) --------------------------

def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns the 16-bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to fp32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


# ---- draws ----------------------------------------------------------------

def draw_mlp(dims: List[int], seed: int, dtype: str, bias_scale: float = 0.0):
    """Weights N(0, 2/fan_in), drawn W1, b1, W2, b2, ... from one generator.

    Returns (W_f32, W_store, bias): W_f32 are the values both sides compute with
    (for bf16 storage: the rounded values, widened); W_store is what the device
    holds (fp32 arrays or uint16 bf16 patterns)."""
    rng = np.random.default_rng(seed)
    W_f32, W_store, bias = [], [], []
    for l in range(len(dims) - 1):
        D, N = dims[l], dims[l + 1]
        w = (rng.standard_normal((N, D), dtype=np.float32) * np.float32(np.sqrt(2.0 / D))).astype(np.float32)
        b = rng.standard_normal(N, dtype=np.float32) * np.float32(bias_scale)
        if dtype == "bf16":
            bits = f32_to_bf16_bits(w)
            W_store.append(bits)
            W_f32.append(bf16_bits_to_f32(bits))
        else:
            W_store.append(w)
            W_f32.append(w)
        bias.append(b.astype(np.float32))
    return W_f32, W_store, bias


def draw_dense_inputs(n: int, D: int, seed: int, law: str) -> np.ndarray:
    rng = np.random.default_rng(seed)
    if law == "u01_half_zero":  # uniform[0,1) with an independent 50 % zero mask
        x = rng.random((n, D), dtype=np.float32)
        keep = rng.random((n, D), dtype=np.float32) < 0.5
        return np.where(keep, x, np.float32(0)).astype(np.float32)
    if law == "relu_normal":    # max(N(0,1), 0)
        x = rng.standard_normal((n, D), dtype=np.float32)
        return np.maximum(x, np.float32(0)).astype(np.float32)
    raise ValueError(law)


def draw_sparse_inputs(n: int, D: int, nnz: int, seed: int):
    """CSR rows with nnz distinct uniform ids (ascending) and log-normal(0,1) values."""
    rng = np.random.default_rng(seed)
    ids = np.empty((n, nnz), dtype=np.uint32)
    for q in range(n):
        ids[q] = np.sort(rng.choice(D, size=nnz, replace=False)).astype(np.uint32)
    vals = np.exp(rng.standard_normal((n, nnz))).astype(np.float32)
    indptr = (np.arange(n + 1, dtype=np.uint64) * np.uint64(nnz))
    return indptr, ids.reshape(-1), vals.reshape(-1)


def draw_mixed_budgets(n: int, seed: int, choices=(500, 1000, 2500, 5000, 10000)) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return np.asarray(choices, dtype=np.uint16)[rng.integers(0, len(choices), size=n)]


# ---- named workloads --------------------------------------------------------

@dataclass
class Workload:
    name: str
    dims: List[int]
    has_act: List[int]
    dtype: str                      # "f32" | "bf16" (weight storage)
    W_f32: List[np.ndarray]
    W_store: List[np.ndarray]
    bias: List[np.ndarray]
    first_sparse: bool
    calib: object                   # dense [n_cal, D0] or CSR triple
    x: object                       # dense [n, D0] or CSR triple
    budget_bp: np.ndarray           # [n] uint16
    K: int = 10
    L: int = 2
    seed: int = 0                   # hash-node sampling seed
    list_cap: int = 0
    budgets_named: Tuple[int, ...] = field(default_factory=tuple)
    free_hash_nodes: bool = False   # hash nodes always active and absent from the lists (Sec. 3.4 variant)

    @property
    def n_queries(self) -> int:
        return int(self.budget_bp.size)

    @property
    def V(self) -> int:
        return 8 if self.dtype == "bf16" else 4


_SPECS = {
    # name: dims, has_act, dtype, w_seed, x_seed, calib_seed, law, n_queries, n_cal, budgets
    "c1": dict(dims=[784, 112, 112, 10], has_act=[1, 1, 0], dtype="f32", w_seed=0, x_seed=1,
               c_seed=101, law="u01_half_zero", n=1024, n_cal=16384, budgets=(1000, 2500, 5000, 10000)),
    "c2": dict(dims=[784, 1024, 1024, 10], has_act=[1, 1, 0], dtype="bf16", w_seed=2, x_seed=12,
               c_seed=102, law="u01_half_zero", n=65536, n_cal=16384, budgets=(500, 1000, 2500, 5000, 10000)),
    "c3": dict(dims=[100000, 128, 200000], has_act=[0, 1], dtype="f32", w_seed=20, x_seed=21,
               c_seed=103, law="sparse75", n=256, n_cal=16384, budgets=(100, 500, 1000)),
    # like c3 with a 1,000,000-node output layer (512 MB of fp32 rows, four times the L2): the gathered rows
    # come from HBM, not from cache.  Lists are capped at 10,000 entries (1 % of the layer).
    "c3xl": dict(dims=[100000, 128, 1000000], has_act=[0, 1], dtype="f32", w_seed=22, x_seed=23,
                 c_seed=106, law="sparse75", n=256, n_cal=2048, budgets=(10, 50, 100), list_cap=10000),
    "c4": dict(dims=[4096] + [4096] * 8 + [1000], has_act=[1] * 8 + [0], dtype="bf16", w_seed=3,
               x_seed=31, c_seed=104, law="relu_normal", n=4096, n_cal=8192, budgets=(1000, 2500, 5000)),
    "c5": dict(dims=[2048, 4096, 4096, 1000], has_act=[1, 1, 0], dtype="bf16", w_seed=40, x_seed=41,
               c_seed=105, law="relu_normal", n=8192, n_cal=16384, budgets=(500, 1000, 2500, 5000, 10000)),
}


def load(name: str, n_queries: Optional[int] = None, n_cal: Optional[int] = None,
         budget_bp: Optional[int] = None, list_cap: int = 0, dims: Optional[List[int]] = None,
         free_hash_nodes: bool = False) -> Workload:
    """Draw a named workload.  n_queries / n_cal shrink the query and calibration
    sets (same laws, same seeds); budget_bp gives every query one budget, else
    c5 draws a mixed stream (seed 4) and the others use their first named budget.
    dims overrides the layer widths (scaled-down copies for quick checks)."""
    s = _SPECS[name]
    dims_ = list(dims) if dims is not None else list(s["dims"])
    has_act = list(s["has_act"])
    assert len(dims_) == len(s["dims"])
    n = int(n_queries if n_queries is not None else s["n"])
    nc = int(n_cal if n_cal is not None else s["n_cal"])
    W_f32, W_store, bias = draw_mlp(dims_, s["w_seed"], s["dtype"])
    first_sparse = s["law"] == "sparse75"
    if first_sparse:
        x = draw_sparse_inputs(n, dims_[0], 75, s["x_seed"])
        calib = draw_sparse_inputs(nc, dims_[0], 75, s["c_seed"])
    else:
        x = draw_dense_inputs(n, dims_[0], s["x_seed"], s["law"])
        calib = draw_dense_inputs(nc, dims_[0], s["c_seed"], s["law"])
    if budget_bp is not None:
        bp = np.full(n, int(budget_bp), dtype=np.uint16)
    elif name == "c5":
        bp = draw_mixed_budgets(n, 4)
    else:
        bp = np.full(n, s["budgets"][0], dtype=np.uint16)
    return Workload(name=name, dims=dims_, has_act=has_act, dtype=s["dtype"], W_f32=W_f32,
                    W_store=W_store, bias=bias, first_sparse=first_sparse, calib=calib, x=x,
                    budget_bp=bp, seed=s["w_seed"] + 1000, list_cap=list_cap or s.get("list_cap", 0),
                    budgets_named=tuple(s["budgets"]), free_hash_nodes=bool(free_hash_nodes))
