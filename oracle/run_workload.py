"""The CPU oracle applied to a workload description (test infrastructure, like the rest of this
folder: only tests, the smoke check and the benchmark's CPU-baseline legs may use it).

A workload is any object with the attributes of `paper_2204_08400_b200.workloads.Workload`
(dims, has_act, W_f32, bias, V, K, L, list_cap, first_sparse, free_hash_nodes, calib, x, seed);
nothing of the CUDA library is imported here."""
import numpy as np

from . import oracle as orc


def oracle_model(wl, n_cal=None, hash_nodes_override=None) -> orc.OracleModel:
    """Algorithm 1 on the workload's calibration rows (the first n_cal of them)."""
    m = orc.OracleModel(wl.dims, wl.has_act, wl.W_f32, wl.bias, V=wl.V, K=wl.K, L=wl.L,
                        list_cap=wl.list_cap, first_sparse=wl.first_sparse, free_hash_nodes=wl.free_hash_nodes)
    if wl.first_sparse:
        ip, ids, vals = wl.calib
        if n_cal is not None:
            ip = ip[: n_cal + 1]
            ids, vals = ids[: int(ip[-1])], vals[: int(ip[-1])]
        m.build(calib_csr=(ip, ids, vals), seed=wl.seed, hash_override=hash_nodes_override)
    else:
        c = wl.calib if n_cal is None else wl.calib[:n_cal]
        m.build(calib_dense=c, seed=wl.seed, hash_override=hash_nodes_override)
    return m


def take_queries(wl, idx):
    """Inputs of the selected queries (dense rows or a CSR slice)."""
    idx = np.asarray(idx)
    if wl.first_sparse:
        ip, ids, vals = wl.x
        lens = (ip[idx + 1] - ip[idx]).astype(np.int64)
        nip = np.zeros(idx.size + 1, np.uint64)
        nip[1:] = np.cumsum(lens)
        sel = np.concatenate([np.arange(int(ip[i]), int(ip[i + 1])) for i in idx]) if idx.size else np.zeros(0, np.int64)
        return (nip, ids[sel], vals[sel])
    return wl.x[idx]


def oracle_run(m, wl, x, bp, mode=orc.CANON32):
    """The SLO-aware forward pass (Sec. 3.3) of queries x at budgets bp."""
    if wl.first_sparse:
        return m.run(bp, x_csr=x, mode=mode)
    return m.run(bp, x_dense=x, mode=mode)
