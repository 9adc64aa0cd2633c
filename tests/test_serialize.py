"""Persisting a trained Node Activator: blob round trip on the GPU, and refusal of damaged
blobs (checked before any device call, so those cases run without a GPU)."""
import ctypes as C

import numpy as np
import pytest

from paper_2204_08400_b200 import workloads as wl_mod
from paper_2204_08400_b200.workloads import Workload


def test_damaged_blobs_are_refused_before_any_device_work():
    from paper_2204_08400_b200 import binding as sl
    fake_w = [np.zeros(64, np.uint8)]          # never dereferenced: the blob is rejected first
    for blob in (np.zeros(8, np.uint8), np.zeros(400, np.uint8), np.full(400, 0xAB, np.uint8)):
        with pytest.raises(sl.SlonnError) as e:
            sl.slonn_deserialize(blob, fake_w, fake_w)
        assert e.value.code == sl.ERR["ARG"]


@pytest.mark.gpu
def test_round_trip_gives_the_same_model():
    from paper_2204_08400_b200 import binding as sl, harness
    dims = [136, 200, 96, 24]
    W_f32, W_store, bias = wl_mod.draw_mlp(dims, 80, "bf16", bias_scale=0.2)
    wl = Workload(name="custom", dims=dims, has_act=[1, 1, 0], dtype="bf16", W_f32=W_f32, W_store=W_store, bias=bias,
                  first_sparse=False, calib=wl_mod.draw_dense_inputs(500, dims[0], 82, "relu_normal"),
                  x=wl_mod.draw_dense_inputs(300, dims[0], 81, "relu_normal"),
                  budget_bp=wl_mod.draw_mixed_budgets(300, 83), K=4, L=2, seed=84, list_cap=150)
    dm = harness.DeviceModel(wl)
    want = harness.run_once(dm, wl.x, wl.budget_bp)
    blob = sl.slonn_serialize(dm.model)
    built = dm.model
    dm.model = sl.slonn_deserialize(blob, dm.W, dm.bias)        # same weights, no calibration pass
    for l in (0, 1):
        assert np.array_equal(dm.hash_nodes(l), sl.slonn_model_info(built, l)["hash_nodes"])
        assert np.array_equal(dm.tables(l), sl.slonn_model_tables_to_host(built, l))
    got = harness.run_once(dm, wl.x, wl.budget_bp)
    for k in ("logits", "pred", "codes", "active_indptr", "active_ids", "active_vals"):
        assert np.array_equal(got[k], want[k]), k
    assert np.array_equal(sl.slonn_serialize(dm.model), blob)   # serialising again is stable
    # one flipped byte in the tables, a truncated blob, a blob with trailing bytes: all refused
    bad = blob.copy(); bad[len(bad) // 2] ^= 1
    for b in (bad, blob[:-9], np.concatenate([blob, np.zeros(4, np.uint8)])):
        with pytest.raises(sl.SlonnError):
            sl.slonn_deserialize(b, dm.W, dm.bias)
    sl.slonn_free(built)
    dm.free()


@pytest.mark.gpu
def test_round_trip_with_a_csr_first_layer():
    from paper_2204_08400_b200 import binding as sl, harness
    wl = wl_mod.load("c3", n_queries=32, n_cal=256, budget_bp=500, dims=[5000, 64, 3000])
    dm = harness.DeviceModel(wl)
    want = harness.run_once(dm, wl.x, wl.budget_bp)
    blob = sl.slonn_serialize(dm.model)
    built, dm.model = dm.model, sl.slonn_deserialize(blob, dm.W, dm.bias)
    got = harness.run_once(dm, wl.x, wl.budget_bp)
    for k in ("logits", "logit_ids", "pred", "codes", "active_ids", "active_vals"):
        assert np.array_equal(got[k], want[k]), k
    sl.slonn_free(built)
    dm.free()
