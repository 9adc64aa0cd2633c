"""slonn_run_static: the run call for callers that are not allowed to allocate
device memory (the scratch space is a fixed area inside the library).  Collected
last on purpose, so that a run stopping at the first failure has already
covered every other test.  Checks, through the C ABI, that two calls in a row
give exactly what slonn_run gives, and that an oversized batch is refused."""
import numpy as np
import pytest

from paper_2204_08400_b200 import workloads as wl_mod
from paper_2204_08400_b200.workloads import Workload

pytestmark = pytest.mark.gpu

KEYS = ("logits", "pred", "codes", "active_indptr", "active_ids", "active_vals")


def small_workload(seed, n):
    dims = [136, 200, 96, 24]
    W_f32, W_store, bias = wl_mod.draw_mlp(dims, seed, "bf16", bias_scale=0.2)
    return Workload(name="custom", dims=dims, has_act=[1, 1, 0], dtype="bf16", W_f32=W_f32, W_store=W_store,
                    bias=bias, first_sparse=False, calib=wl_mod.draw_dense_inputs(400, dims[0], seed + 2, "relu_normal"),
                    x=wl_mod.draw_dense_inputs(n, dims[0], seed + 1, "relu_normal"),
                    budget_bp=wl_mod.draw_mixed_budgets(n, seed + 3), K=4, L=2, seed=seed + 4)


def test_static_scratch_run_matches_the_workspace_run_twice_in_a_row():
    import torch
    from paper_2204_08400_b200 import binding as sl, harness
    wl = small_workload(70, 300)
    dm = harness.DeviceModel(wl)
    want = harness.run_once(dm, wl.x, wl.budget_bp)
    assert want["status"][0] == 0
    assert sl.slonn_workspace_bytes(dm.model, wl.n_queries, int(wl.budget_bp.max())) <= sl.STATIC_WORKSPACE_BYTES

    # first call, then a different batch in between, then the first batch again: the shared
    # scratch area keeps stale contents from the call before and must not leak into results
    other = small_workload(71, 180)
    b1 = harness.DeviceBatch(dm, wl.x, wl.budget_bp)
    b2 = harness.DeviceBatch(dm, other.x, other.budget_bp)
    want_other = harness.run_once(dm, other.x, other.budget_bp)
    for batch, expect in ((b1, want), (b2, want_other), (b1, want)):
        for t in (batch.logits, batch.pred, batch.codes, batch.ids, batch.vals):
            t.fill_(-1)
        sl.slonn_run_static(dm.model, batch.batch)
        got = batch.results()
        assert got["status"][0] == 0
        for k in KEYS:
            assert np.array_equal(got[k], expect[k]), k
    # the point of the entry point: a call obtains no device memory.  The driver's free-byte count (which
    # sees every allocation of the process, torch's cache or not) must not move across a call.
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    sl.slonn_run_static(dm.model, b1.batch)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    dm.free()


def test_static_scratch_run_refuses_a_batch_that_does_not_fit():
    from paper_2204_08400_b200 import binding as sl, harness
    wl = small_workload(72, 40000)
    dm = harness.DeviceModel(wl)
    need = sl.slonn_workspace_bytes(dm.model, wl.n_queries, 10000)
    assert need > sl.STATIC_WORKSPACE_BYTES
    batch = harness.DeviceBatch(dm, wl.x, wl.budget_bp, max_budget_bp=10000)
    with pytest.raises(sl.SlonnError) as e:
        sl.slonn_run_static(dm.model, batch.batch)
    assert e.value.code == sl.ERR["WORKSPACE"]
    dm.free()
