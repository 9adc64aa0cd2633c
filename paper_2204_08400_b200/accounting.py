"""Weight bytes a launch of the library has to touch, counted on the host from the launch records of
`slonn_run_traced` and the batch's budgets (host logic only: nothing here runs on the device and nothing
here is part of the forward pass).

Per query and layer l (input width D, N nodes, weight element size s, K*L = H hash functions, L tables,
node ids of 2 bytes up to 65,536 nodes, else 4):

    hash rows       H * D * s          when whole hash rows are read (dense input, or a list scattered
                                       into a dense vector), H * B_in * s when only the list entries are
    bucket lists    L * B_out * idbytes
    selected nodes  B_out * D * s      row form: every selected weight row whole
                    B_out * B_in * s   input-stationary form: selected nodes x input list entries
    CSR first layer nnz * N * s        one row of the transposed weights per nonzero

with B_out the node count of the query's budget in this layer (N without activator) and B_in the length of
the list the layer below hands over (D when the input is dense).  Three totals are kept per launch:

    as_run         the form each layer actually took (what the kernel had to load)
    algorithmic    the sparse count everywhere (B_out * B_in, H * B_in): the least any form could load
    row_granular   whole rows everywhere
"""
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

KERNEL_OF_STAGE = {
    "plan": "plan_kernels", "hash_select": "hash_select_kernel", "gather_dot": "gather_dot_kernel",
    "sparse_first": "sparse_first_layer_kernel", "argmax": "argmax_kernel", "fused": "fused_network_kernel",
    "dense_tc": "dense_tc_kernel", "cluster": "cluster_network_kernel", "gather_cols": "gather_cols_kernel",
    "layer_cols": "layer_cols_kernel", "full_rows": "full_rows_kernel", "group_rows": "group_rows_kernel",
}


@dataclass
class NetShape:
    dims: List[int]
    has_act: List[int]
    esz: int                      # bytes per weight element
    K: int
    L: int
    first_sparse: bool = False
    pre: int = 0                  # hash nodes that are always active (0, or K*L for such models)

    @classmethod
    def of(cls, wl) -> "NetShape":
        return cls(list(wl.dims), list(wl.has_act), 2 if wl.dtype == "bf16" else 4, wl.K, wl.L,
                   bool(wl.first_sparse), wl.K * wl.L if wl.free_hash_nodes else 0)

    @property
    def n_layers(self) -> int:
        return len(self.dims) - 1


def layer_nodes(bp: np.ndarray, N: int, pre: int = 0) -> np.ndarray:
    """Nodes a layer of N nodes computes at budget bp (basis points): nearest whole node, at least one."""
    B = np.clip((bp.astype(np.int64) * N + 5000) // 10000, 1, N)
    if pre:
        B = np.minimum(B, N - pre) + pre
    return B


def _layer_terms(sh: NetShape, l: int, bp: np.ndarray):
    D, N, s = sh.dims[l], sh.dims[l + 1], sh.esz
    act = bool(sh.has_act[l])
    list_in = l > 0 and bool(sh.has_act[l - 1])
    b_out = layer_nodes(bp, N, sh.pre) if act else np.full(bp.size, N, np.int64)
    b_in = layer_nodes(bp, D, sh.pre) if list_in else np.full(bp.size, D, np.int64)
    H = sh.K * sh.L if act else 0
    idb = 2 if N <= 65536 else 4
    return dict(
        hash_row=H * D * s * np.ones(bp.size, np.int64), hash_alg=H * b_in * s,
        lists=(sh.L * b_out * idb) if act else np.zeros(bp.size, np.int64),
        rows_row=b_out * D * s, rows_alg=b_out * b_in * s, list_in=list_in, act=act)


def served(rec: dict, bps: np.ndarray) -> np.ndarray:
    """Mask of the queries a launch serves."""
    m = (bps >= rec["bp_lo"]) & (bps <= rec["bp_hi"])
    if rec["skips_full"]:
        m &= bps != 10000
    return m


def launch_bytes(sh: NetShape, rec: dict, bps: Sequence[int], x_nnz: Optional[np.ndarray] = None) -> dict:
    """Totals over the queries the launch serves: as_run / algorithmic / row_granular bytes, flops (tensor-core
    launches) and the number of queries."""
    bps = np.asarray(bps).astype(np.int64)
    m = served(rec, bps)
    bp = bps[m]
    out = dict(as_run=0, algorithmic=0, row_granular=0, flops=0.0, queries=int(m.sum()))
    if bp.size == 0:
        return out
    stage = rec["stage"]
    layers = range(sh.n_layers) if rec["layer"] is None else [rec["layer"]]
    for l in layers:
        if stage in ("plan", "argmax"):
            break
        if l == 0 and sh.first_sparse:
            if stage == "sparse_first":
                nnz = np.asarray(x_nnz, np.int64)[m] if x_nnz is not None else np.zeros(bp.size, np.int64)
                b = int(nnz.sum()) * sh.dims[1] * sh.esz
                out["as_run"] += b; out["algorithmic"] += b; out["row_granular"] += b
            continue
        t = _layer_terms(sh, l, bp)
        if stage == "dense_tc":
            out["flops"] += 2.0 * bp.size * sh.dims[l] * sh.dims[l + 1]
            continue
        if stage == "sparse_first":
            continue
        alg = row = run = 0
        hashes = stage in ("hash_select", "layer_cols", "fused", "cluster")
        nodes = stage in ("gather_dot", "gather_cols", "layer_cols", "full_rows", "group_rows", "fused", "cluster")
        cols = np.zeros(bp.size, bool)
        if stage in ("gather_cols", "layer_cols"):
            cols[:] = True
        elif stage == "fused" and rec["cols_bp"] and t["act"] and t["list_in"]:
            cols = bp <= rec["cols_bp"]
        if hashes and t["act"]:
            alg += int((t["hash_alg"] + t["lists"]).sum())
            row += int((t["hash_row"] + t["lists"]).sum())
            run += int((np.where(cols, t["hash_alg"], t["hash_row"]) + t["lists"]).sum())
        if nodes:
            alg += int(t["rows_alg"].sum())
            row += int(t["rows_row"].sum())
            run += int(np.where(cols, t["rows_alg"], t["rows_row"]).sum())
        out["as_run"] += run; out["algorithmic"] += alg; out["row_granular"] += row
    return out


def kernel_name(sh: NetShape, rec: dict) -> str:
    """The kernel behind a record (rows of at most one 512-byte round take the short-row gather)."""
    if rec["stage"] == "gather_dot" and rec["layer"] is not None and sh.dims[rec["layer"]] * sh.esz <= 512:
        return "gather_short_kernel"
    return KERNEL_OF_STAGE[rec["stage"]]


def per_kernel(sh: NetShape, records: List[dict], bps, x_nnz=None) -> dict:
    """Launch records of ONE step grouped by kernel: launches, ms and the three byte totals."""
    acc = {}
    for r in records:
        k = kernel_name(sh, r)
        b = launch_bytes(sh, r, bps, x_nnz)
        a = acc.setdefault(k, dict(launches=0, ms=0.0, as_run=0, algorithmic=0, row_granular=0, flops=0.0))
        a["launches"] += 1
        a["ms"] += r["ms"]
        for key in ("as_run", "algorithmic", "row_granular", "flops"):
            a[key] += b[key]
    return acc


def step_bytes(sh: NetShape, bps, x_nnz=None) -> dict:
    """Bytes of a whole step from the formulas alone (no records): every layer row-wise, and every layer
    in the sparse count."""
    whole = dict(stage="cluster", layer=None, bp_lo=0, bp_hi=10000, skips_full=False, cols_bp=0)
    b = launch_bytes(sh, whole, bps, x_nnz)
    if sh.first_sparse:
        first = launch_bytes(sh, dict(whole, stage="sparse_first", layer=0), bps, x_nnz)
        for k in ("as_run", "algorithmic", "row_granular"):
            b[k] += first[k]
    return dict(algorithmic=b["algorithmic"], row_granular=b["row_granular"])
