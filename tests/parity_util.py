"""Helpers of the GPU parity tests: build the same model on both sides and
compare element by element.  The GPU results come through the C ABI; the
expected values come from the CPU oracle only."""
import numpy as np

from oracle import oracle as orc
from oracle.run_workload import oracle_model, oracle_run, take_queries  # noqa: F401 (re-exported)
from paper_2204_08400_b200.workloads import Workload

TOL = {"f32": 1e-5, "bf16": 2e-2}   # max relative logit error against the fp64 oracle


def assert_build_parity(dm, om, wl: Workload):
    for l in range(len(wl.dims) - 1):
        if not wl.has_act[l]:
            continue
        assert np.array_equal(dm.hash_nodes(l), om.hash_nodes(l)), f"hash nodes of layer {l}"
        got = dm.tables(l).astype(np.uint32)
        want = om.rank(l)
        assert got.shape == want.shape, f"table shape of layer {l}"
        assert np.array_equal(got, want), f"bucket contents of layer {l}"


def assert_run_parity(g: dict, o32: dict, o64: dict, wl: Workload, n_act: int, last_budgeted: bool):
    """g: GPU results; o32 / o64: oracle in its fp32-contract and fp64 modes, same queries."""
    n = o32["pred"].size
    assert g["status"][0] == 0, f"device status {g['status']}"
    assert np.array_equal(g["codes"], o32["codes"]), "hash codes"
    assert np.array_equal(g["active_indptr"], o32["active_indptr"]), "active offsets"
    assert np.array_equal(g["active_ids"], o32["active_ids"]), "active sets"
    assert np.array_equal(g["pred"], o32["pred"]), "argmax"
    assert np.array_equal(g["active_vals"], o32["active_vals"]), "activations (same summation order)"
    stride = o32["logit_stride"]
    if last_budgeted:
        ip = o32["active_indptr"].astype(np.int64)
        for q in range(n):
            B = int(ip[q * n_act + n_act] - ip[q * n_act + n_act - 1])
            assert np.array_equal(g["logit_ids"][q, :B], o32["logit_ids"][q, :B])
            assert np.array_equal(g["logits"][q, :B], o32["logits"][q, :B])
    else:
        assert np.array_equal(g["logits"][:, :stride], o32["logits"]), "logits (same summation order)"
    # tolerance against the fp64 definition, on queries where fp32 and fp64 take the same decisions
    same = np.all(o32["codes"] == o64["codes"], axis=(1, 2)) if n_act else np.ones(n, bool)
    tol = TOL[wl.dtype]
    worst = 0.0
    ip = o32["active_indptr"].astype(np.int64)
    for q in np.nonzero(same)[0]:
        if last_budgeted:
            B = int(ip[q * n_act + n_act] - ip[q * n_act + n_act - 1])
            a, b = g["logits"][q, :B].astype(np.float64), o64["logits"][q, :B]
        else:
            a, b = g["logits"][q, :stride].astype(np.float64), o64["logits"][q]
        worst = max(worst, float(np.max(np.abs(a - b)) / max(np.max(np.abs(b)), 1e-30)))
    assert worst <= tol, f"max relative logit error {worst} > {tol}"
    return {"decision_disagreements": int((~same).sum()), "max_rel_err": worst}
