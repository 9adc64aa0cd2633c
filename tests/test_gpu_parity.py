"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on
the same seeded inputs.  Integer results (hash codes, bucket contents, active
sets, argmax) must be bit-exact; logits within 1e-5 (fp32 weights) / 2e-2 (bf16
weights) of the fp64 oracle, relative to the largest logit of the query."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2204_08400_b200 import workloads as wl_mod
from paper_2204_08400_b200.workloads import Workload
from parity_util import assert_build_parity, assert_run_parity, oracle_model, oracle_run, take_queries

pytestmark = pytest.mark.gpu


def custom_workload(seed, dims, has_act, dtype, n, n_cal, K, L, law="relu_normal", bias_scale=0.2,
                    list_cap=0, budgets=(500, 1000, 2500, 5000, 10000)):
    W_f32, W_store, bias = wl_mod.draw_mlp(dims, seed, dtype, bias_scale=bias_scale)
    x = wl_mod.draw_dense_inputs(n, dims[0], seed + 1, law)
    calib = wl_mod.draw_dense_inputs(n_cal, dims[0], seed + 2, law)
    bp = wl_mod.draw_mixed_budgets(n, seed + 3, budgets)
    return Workload(name="custom", dims=list(dims), has_act=list(has_act), dtype=dtype, W_f32=W_f32,
                    W_store=W_store, bias=bias, first_sparse=False, calib=calib, x=x, budget_bp=bp,
                    K=K, L=L, seed=seed + 4, list_cap=list_cap)


def kernel_paths(wl):
    """Both kernel families where the network fits the one-warp-per-query kernel, else the staged one."""
    fused_ok = (not wl.first_sparse) and max(wl.dims[:-1]) <= 1024 and max(wl.dims[1:]) <= 4096
    cluster_ok = (not wl.first_sparse) and max(wl.dims) <= 8192 and wl.n_queries <= 600
    return (1,) + ((2, 4) if fused_ok else ()) + ((3,) if cluster_ok else ())   # 4: one block of four warps per query


def check(wl, n_cal=None, sample=None, expect_build=True, models=None):
    """models: a (device model, oracle model) pair built earlier from the same weights and calibration rows
    (the tables do not depend on the budgets); it is then neither compared again nor freed here."""
    from paper_2204_08400_b200 import binding as sl, harness
    if models is None:
        dm = harness.DeviceModel(wl, n_cal=n_cal)
        om = oracle_model(wl, n_cal=n_cal)
        if expect_build:
            assert_build_parity(dm, om, wl)
    else:
        dm, om = models
    n_act = sum(wl.has_act)
    if sample is None:
        x, bp = wl.x, wl.budget_bp
    else:
        x, bp = take_queries(wl, sample), wl.budget_bp[sample]
    o32 = oracle_run(om, wl, x, bp, orc.CANON32)
    o64 = oracle_run(om, wl, x, bp, orc.REF64)
    info = None
    for path in kernel_paths(wl):
        # the per-stage and one-warp-per-query kernels evaluate a sparse-input layer row-wise or
        # input-wise: library's choice, then each kind forced for the whole batch
        # (and, for the per-stage row kernels, every query in a block of its own instead of four per block)
        for flags in ((0, sl.FLAG_ROW_KERNELS, sl.FLAG_COLUMN_KERNELS) + ((sl.FLAG_ROW_KERNELS | sl.FLAG_UNGROUPED_ROWS,) if path == 1 else ())
                      if path in (1, 2) else (0,)):
            g = harness.run_once(dm, wl.x, wl.budget_bp, kernel_path=path, flags=flags)
            if sample is not None:
                g = slice_results(g, sample, n_act)
            info = assert_run_parity(g, o32, o64, wl, n_act, bool(wl.has_act[-1]))
    # the configuration the benchmark times: the library picks the kernels and the caller asks for
    # logits and predictions only (no active lists, so some paths skip the planning launches)
    g = harness.run_once(dm, wl.x, wl.budget_bp)
    b = harness.DeviceBatch(dm, wl.x, wl.budget_bp, full_outputs=False)
    b.run()
    lean = b.results()
    assert lean["status"][0] == 0
    assert np.array_equal(lean["pred"], g["pred"]), "argmax without lists"
    if wl.has_act[-1]:
        ip = g["active_indptr"].astype(np.int64)
        for q in (range(wl.n_queries) if sample is None else sample):
            B = int(ip[q * n_act + n_act] - ip[q * n_act + n_act - 1])
            assert np.array_equal(lean["logits"][q, :B], g["logits"][q, :B]), "logits without lists"
    else:
        assert np.array_equal(lean["logits"], g["logits"]), "logits without lists"
    if sample is not None:
        g = slice_results(g, sample, n_act)
    assert_run_parity(g, o32, o64, wl, n_act, bool(wl.has_act[-1]))
    if models is None:
        dm.free()
    return info


def build_both(wl, n_cal=None):
    """Device model and oracle model of a workload, bucket contents compared."""
    from paper_2204_08400_b200 import harness
    dm = harness.DeviceModel(wl, n_cal=n_cal)
    om = oracle_model(wl, n_cal=n_cal)
    assert_build_parity(dm, om, wl)
    return dm, om


def slice_results(g, idx, n_act):
    """Restrict full-batch GPU results to the sampled queries (CSR payload re-packed)."""
    idx = np.asarray(idx)
    ip = g["active_indptr"].astype(np.int64)
    out = {"status": g["status"], "logits": g["logits"][idx], "pred": g["pred"][idx],
           "codes": g["codes"][idx], "logit_stride": g["logit_stride"]}
    if "logit_ids" in g:
        out["logit_ids"] = g["logit_ids"][idx]
    nip = [0]
    ids, vals = [], []
    for q in idx:
        for a in range(n_act):
            s, e = ip[q * n_act + a], ip[q * n_act + a + 1]
            ids.append(g["active_ids"][s:e]); vals.append(g["active_vals"][s:e])
            nip.append(nip[-1] + int(e - s))
    out["active_indptr"] = np.asarray(nip, dtype=np.uint64)
    out["active_ids"] = np.concatenate(ids) if ids else np.zeros(0, np.uint32)
    out["active_vals"] = np.concatenate(vals) if vals else np.zeros(0, np.float32)
    return out


# ---- small shapes spanning several tiles and ragged tails ----------------------

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_small_mlp_mixed_budgets(dtype):
    wl = custom_workload(50, [136, 200, 96, 24], [1, 1, 0], dtype, n=300, n_cal=700, K=4, L=2)
    check(wl)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_three_tables_and_output_activator(dtype):
    wl = custom_workload(51, [72, 160, 328], [1, 1], dtype, n=120, n_cal=500, K=3, L=3,
                         budgets=(100, 700, 3300, 10000))
    check(wl)


def test_single_table_single_bit():
    wl = custom_workload(52, [40, 64, 8], [1, 0], "f32", n=64, n_cal=100, K=1, L=1)
    check(wl)


def test_list_cap():
    wl = custom_workload(53, [64, 256, 16], [1, 0], "bf16", n=200, n_cal=600, K=5, L=2, list_cap=70,
                         budgets=(100, 1000, 2500, 10000))   # B = 3, 26, 64, 256 (all)
    check(wl)


def test_no_activators_is_the_dense_network():
    wl = custom_workload(54, [96, 128, 40], [0, 0], "f32", n=77, n_cal=10, K=2, L=1)
    check(wl)


# ---- the benchmark shapes -------------------------------------------------------

def test_c1_full():
    for bp in (1000, 2500, 5000, 10000):
        wl = wl_mod.load("c1", budget_bp=bp, n_cal=4096)
        check(wl, expect_build=(bp == 1000))


def test_c2_reduced_queries_all_budgets():
    for bp in (500, 1000, 2500, 5000, 10000):
        wl = wl_mod.load("c2", n_queries=1024, n_cal=2048, budget_bp=bp)
        check(wl, expect_build=(bp == 500))


def test_c3_narrow_output():
    # same structure as the wide-output net with a 20,000-node output layer
    for bp in (100, 500, 1000):
        wl = wl_mod.load("c3", n_queries=64, n_cal=512, budget_bp=bp, dims=[100000, 128, 20000])
        check(wl, expect_build=(bp == 100))


def test_c4_narrow_batches():
    for n in (1, 64):
        wl = wl_mod.load("c4", n_queries=n, n_cal=1024, budget_bp=2500, dims=[512] + [512] * 8 + [104])
        check(wl, expect_build=(n == 1))


def test_c5_mixed_budgets_reduced():
    wl = wl_mod.load("c5", n_queries=512, n_cal=1024, dims=[512, 1024, 1024, 200])
    assert len(set(wl.budget_bp.tolist())) == 5
    check(wl)


# ---- full sizes, in the launch configuration the benchmark times, on sampled queries ----

def with_budget(wl, bp):
    import dataclasses
    return dataclasses.replace(wl, budget_bp=np.full(wl.n_queries, bp, np.uint16))


def test_c2_full_size_every_named_budget_sampled():
    wl = wl_mod.load("c2", budget_bp=1000)                      # 65,536 queries, 16,384 calibration rows
    sample = np.unique(np.linspace(0, wl.n_queries - 1, 192).astype(np.int64))
    models = build_both(wl)
    for bp in (1000, 500, 2500, 5000, 10000):
        info = check(with_budget(wl, bp), sample=sample, models=models)
        assert info["decision_disagreements"] <= 2
    models[0].free()


def test_c5_full_widths_mixed_budgets_sampled():
    wl = wl_mod.load("c5", n_queries=8192, n_cal=512)            # one batch of the mixed-budget stream
    sample = np.unique(np.linspace(0, wl.n_queries - 1, 48).astype(np.int64))
    check(wl, n_cal=512, sample=sample)


def test_c5_full_widths_single_budgets_sampled():
    # the budget sweep of the benchmark: 8192 queries at one budget each
    wl = wl_mod.load("c5", n_queries=8192, n_cal=512, budget_bp=500)
    sample = np.unique(np.linspace(0, wl.n_queries - 1, 16).astype(np.int64))
    models = build_both(wl, n_cal=512)
    for bp in (500, 1000, 2500, 5000, 10000):
        check(with_budget(wl, bp), sample=sample, models=models)
    models[0].free()


def test_c4_full_widths_batch_sizes_and_budgets_sampled():
    import dataclasses
    big = wl_mod.load("c4", n_queries=4096, n_cal=192, budget_bp=1000)   # the batch size the benchmark times
    models = build_both(big, n_cal=192)
    for n, k, budgets in ((1, 1, (1000, 2500, 5000)), (64, 8, (1000, 2500, 5000)), (4096, 16, (1000, 2500, 5000))):
        wl = dataclasses.replace(big, x=big.x[:n], budget_bp=big.budget_bp[:n])
        sample = np.unique(np.linspace(0, n - 1, k).astype(np.int64))
        for bp in budgets:
            check(with_budget(wl, bp), sample=sample, models=models)
    models[0].free()


def test_c3_full_width_output_layer_sampled():
    # 200,000 output nodes; lists cut at the largest budget the workload names (10 %)
    wl = wl_mod.load("c3", n_queries=256, n_cal=256, budget_bp=1000, list_cap=20000)
    sample = np.arange(0, 256, 32)
    models = build_both(wl, n_cal=256)
    for bp in (1000, 500, 100):
        check(with_budget(wl, bp), sample=sample, models=models)
    models[0].free()


def test_c3_full_width_complete_rankings_sampled():
    # the tables the benchmark builds: every bucket list a complete ranking of the 200,000 nodes (1.6 GB)
    wl = wl_mod.load("c3", n_queries=256, n_cal=256, budget_bp=1000)
    assert wl.list_cap == 0
    sample = np.arange(5, 256, 50)
    models = build_both(wl, n_cal=256)
    for bp in (100, 1000):
        check(with_budget(wl, bp), sample=sample, models=models)
    models[0].free()


# ---- edge cases -----------------------------------------------------------------

def test_empty_batch_and_single_query():
    from paper_2204_08400_b200 import harness
    wl = custom_workload(55, [32, 64, 8], [1, 0], "f32", n=1, n_cal=50, K=2, L=2)
    dm = harness.DeviceModel(wl)
    g = harness.run_once(dm, wl.x[:0], wl.budget_bp[:0], max_budget_bp=10000)
    assert g["status"][0] == 0 and g["pred"].size == 0
    dm.free()
    check(wl)


def test_one_node_budget():
    wl = custom_workload(56, [48, 96, 16], [1, 0], "bf16", n=40, n_cal=200, K=3, L=2, budgets=(1, 50))
    check(wl)


def test_invalid_budget_is_reported_not_fatal():
    from paper_2204_08400_b200 import harness
    wl = custom_workload(57, [32, 64, 8], [1, 0], "f32", n=16, n_cal=80, K=2, L=2, budgets=(2500,))
    dm = harness.DeviceModel(wl)
    for path in (1, 2, 3, 4):
        bp = wl.budget_bp.copy()
        bp[5] = 0
        g = harness.run_once(dm, wl.x, bp, max_budget_bp=5000, kernel_path=path)
        assert g["status"][0] == 5 and g["status"][1] == 5     # SLONN_ERR_BUDGET at query 5
        bp[5] = 2500
        g = harness.run_once(dm, wl.x, bp, max_budget_bp=5000, kernel_path=path)
        assert g["status"][0] == 0
    dm.free()


@pytest.mark.parametrize("last_budgeted", [False, True])
def test_one_warp_per_query_kernel_without_active_lists(last_budgeted):
    # a caller that asks for logits and predictions only: the one-warp-per-query kernel then runs without
    # the planning launches and derives each layer's node count from the budget itself; results must not
    # change, mixed budgets included, and an invalid budget must still be reported
    from paper_2204_08400_b200 import binding as sl, harness
    wl = custom_workload(75, [72, 160, 120, 24], [1, 1, 1 if last_budgeted else 0], "bf16", n=700, n_cal=256, K=3, L=2,
                         budgets=(700, 1000, 4000, 10000))
    dm = harness.DeviceModel(wl)
    for flags in (0, sl.FLAG_ROW_KERNELS, sl.FLAG_COLUMN_KERNELS):
        full = harness.run_once(dm, wl.x, wl.budget_bp, kernel_path=2, flags=flags)
        b = harness.DeviceBatch(dm, wl.x, wl.budget_bp, full_outputs=False, kernel_path=2, flags=flags)
        b.run()
        g = b.results()
        assert g["status"][0] == 0
        assert np.array_equal(g["pred"], full["pred"])
        if last_budgeted:
            ip = full["active_indptr"].astype(np.int64)
            for q in range(wl.n_queries):
                B = int(ip[q * 3 + 3] - ip[q * 3 + 2])
                assert np.array_equal(g["logits"][q, :B], full["logits"][q, :B])
                assert np.array_equal(g["logit_ids"][q, :B], full["logit_ids"][q, :B])
        else:
            assert np.array_equal(g["logits"], full["logits"])
    bp = wl.budget_bp.copy()
    bp[11] = 0
    b = harness.DeviceBatch(dm, wl.x, bp, max_budget_bp=10000, full_outputs=False, kernel_path=2)
    b.run()
    st = b.results()["status"]
    assert st[0] == 5 and st[1] == 11     # SLONN_ERR_BUDGET at query 11
    dm.free()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_four_queries_per_block_row_kernel_on_a_budgeted_last_layer(dtype):
    # rows longer than one 512-byte round, 300 queries (75 groups of four, budgets in both grouping classes and
    # below the grouping limit), the last layer budgeted: the grouped row kernel writes logits and their ids by
    # position; a 100 % budget inside a group selects every row
    wl = custom_workload(78, [512, 640, 520], [1, 1], dtype, n=302, n_cal=400, K=4, L=2,
                         budgets=(700, 2500, 3000, 5000, 10000))
    check(wl)


def test_launch_records_cover_the_step_and_name_what_each_launch_serves():
    from paper_2204_08400_b200 import binding as sl, harness
    wl = custom_workload(79, [512, 640, 520, 24], [1, 1, 0], "bf16", n=600, n_cal=300, K=4, L=2,
                         budgets=(700, 3000, 5000, 10000))
    dm = harness.DeviceModel(wl)
    b = harness.DeviceBatch(dm, wl.x, wl.budget_bp, full_outputs=False, kernel_path=sl.PATH_STAGED)
    recs = sl.slonn_run_traced(dm.model, b.batch, b.ws, b.ws_bytes)
    ms, cnt = sl.slonn_run_timed(dm.model, b.batch, b.ws, b.ws_bytes)
    assert b.results()["status"][0] == 0
    assert len(recs) == sum(cnt.values()) and all(r["ms"] > 0 for r in recs)
    for stage in sl.STAGES:
        assert sum(1 for r in recs if r["stage"] == stage) == cnt[stage], stage
    assert [r["stage"] for r in recs][0] == "plan" and recs[-1]["stage"] == "argmax"
    layers = [r["layer"] for r in recs if r["layer"] is not None]
    assert layers == sorted(layers) and set(layers) == {0, 1, 2}
    # every budget of the batch is served exactly once by the node launches of each layer
    for l in (0, 1, 2):
        for bp in (700, 3000, 5000, 10000):
            served = [r for r in recs if r["layer"] == l and r["stage"] in ("gather_dot", "group_rows", "gather_cols", "layer_cols", "full_rows")
                      and r["bp_lo"] <= bp <= r["bp_hi"] and not (r["skips_full"] and bp == 10000)]
            assert len(served) == 1, (l, bp, served)
    dm.free()


def test_full_budget_queries_beside_the_one_warp_per_query_kernel_with_a_budgeted_last_layer():
    # large enough (queries x weights >= 2^32) for the 100 % queries to leave the one-warp-per-query kernel and
    # run four per block; the last layer carries an activator, so the prediction of every other query is an
    # argmax over its own computed logits and must survive the pass that predicts the 100 % ones
    wl = custom_workload(77, [64, 1024, 1024], [1, 1], "bf16", n=4200, n_cal=512, K=4, L=2,
                         budgets=(500, 2500, 10000))
    assert wl.n_queries * (64 * 1024 + 1024 * 1024) >= 2 ** 32
    sample = np.unique(np.linspace(0, wl.n_queries - 1, 160).astype(np.int64))
    assert len(set(wl.budget_bp[sample].tolist())) == 3
    check(wl, sample=sample)


def test_runs_are_deterministic():
    from paper_2204_08400_b200 import harness
    wl = custom_workload(58, [136, 200, 96, 24], [1, 1, 0], "bf16", n=256, n_cal=300, K=4, L=2)
    dm = harness.DeviceModel(wl)
    runs = [harness.run_once(dm, wl.x, wl.budget_bp, kernel_path=p) for p in (1, 1, 2, 2, 3, 3, 4, 4, 0)]
    for b in runs[1:]:
        for k in ("logits", "pred", "codes", "active_ids", "active_vals"):
            assert np.array_equal(runs[0][k], b[k])
    dm.free()


def test_host_buffer_entry_point_matches_device_entry_point():
    import torch
    from paper_2204_08400_b200 import binding as sl, harness
    wl = custom_workload(59, [64, 128, 24], [1, 0], "f32", n=100, n_cal=200, K=3, L=2)
    dm = harness.DeviceModel(wl)
    want = harness.run_once(dm, wl.x, wl.budget_bp)
    n = wl.n_queries
    max_bp = int(wl.budget_bp.max())
    stride = sl.slonn_logit_stride(dm.model, max_bp)
    logits = np.zeros((n, stride), np.float32)
    pred = np.zeros(n, np.uint32)
    status = np.ones(4, np.uint32)
    codes = np.zeros((n, 1, 2), np.uint16)
    nb = sl.slonn_host_workspace_bytes(dm.model, n, max_bp)
    ws = torch.empty(nb, dtype=torch.uint8, device=dm.device)
    hb = sl.make_batch(n, np.ascontiguousarray(wl.budget_bp), logits, status, x_dense=np.ascontiguousarray(wl.x),
                       max_budget_bp=max_bp, pred=pred, codes=codes)
    up, down = sl.slonn_run_host(dm.model, hb, ws, nb)
    assert status[0] == 0
    assert up == wl.x.nbytes + wl.budget_bp.nbytes
    assert down == logits.nbytes + pred.nbytes + codes.nbytes + 16
    assert np.array_equal(logits, want["logits"]) and np.array_equal(pred, want["pred"])
    assert np.array_equal(codes, want["codes"])
    dm.free()


def test_fused_path_refuses_wide_networks():
    from paper_2204_08400_b200 import binding as sl, harness
    wl = custom_workload(60, [2048, 64, 8], [1, 0], "f32", n=4, n_cal=40, K=2, L=2)
    dm = harness.DeviceModel(wl)
    with pytest.raises(sl.SlonnError) as e:
        harness.run_once(dm, wl.x, wl.budget_bp, kernel_path=2)
    assert e.value.code == sl.ERR["DIM"]
    dm.free()


def test_plan_offsets_span_many_tiles():
    # more (query, layer) entries than one plan tile, mixed budgets: offsets must equal the oracle's
    wl = custom_workload(61, [32, 64, 40, 8], [1, 1, 0], "f32", n=5000, n_cal=100, K=2, L=2)
    check(wl)


def test_host_buffer_entry_point_in_pieces_matches_device_entry_point():
    # 10,000 queries: large enough for the two-stream piecewise route of slonn_run_host
    import torch
    from paper_2204_08400_b200 import binding as sl, harness
    wl = custom_workload(62, [64, 128, 24], [1, 0], "bf16", n=10000, n_cal=200, K=3, L=2)
    dm = harness.DeviceModel(wl)
    want = harness.run_once(dm, wl.x, wl.budget_bp)
    n, max_bp = wl.n_queries, int(wl.budget_bp.max())
    stride = sl.slonn_logit_stride(dm.model, max_bp)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    logits = torch.zeros((n, stride), dtype=torch.float32).pin_memory()
    pred = torch.zeros(n, dtype=torch.int32).pin_memory()
    codes = torch.zeros((n, 1, 2), dtype=torch.int16).pin_memory()
    status = torch.ones(4, dtype=torch.int32).pin_memory()
    nb = sl.slonn_host_workspace_bytes(dm.model, n, max_bp)
    ws = torch.empty(nb, dtype=torch.uint8, device=dm.device)
    bp = wl.budget_bp.copy()
    hb = sl.make_batch(n, pin(bp.view(np.int16)), logits, status, x_dense=pin(wl.x), max_budget_bp=max_bp,
                       pred=pred, codes=codes)
    up, down = sl.slonn_run_host(dm.model, hb, ws, nb)
    assert int(status[0]) == 0
    assert up == wl.x.nbytes + bp.nbytes
    assert np.array_equal(logits.numpy(), want["logits"])
    assert np.array_equal(pred.numpy().view(np.uint32), want["pred"])
    assert np.array_equal(codes.numpy().view(np.uint16), want["codes"])
    # an invalid budget in a later piece is reported with its batch-relative query index
    bp[7777] = 0
    hb = sl.make_batch(n, pin(bp.view(np.int16)), logits, status, x_dense=pin(wl.x), max_budget_bp=max_bp, pred=pred)
    sl.slonn_run_host(dm.model, hb, ws, nb)
    assert int(status[0]) == 5 and int(status[1]) == 7777
    dm.free()


def test_slonn_run_replays_from_a_cuda_graph():
    # slonn_run only enqueues work on the caller's stream (no allocation, no host synchronisation),
    # so a serving loop can capture it once and replay it per request
    import torch
    from paper_2204_08400_b200 import harness
    wl = custom_workload(63, [136, 200, 96, 24], [1, 1, 0], "bf16", n=3, n_cal=300, K=4, L=2)
    dm = harness.DeviceModel(wl)
    for path in (1, 2, 3, 4):
        want = harness.run_once(dm, wl.x, wl.budget_bp, kernel_path=path)
        b = harness.DeviceBatch(dm, wl.x, wl.budget_bp, kernel_path=path)
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            b.run(s)                      # first call outside the capture (sets kernel attributes)
            s.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                b.run(torch.cuda.current_stream())
            for t in (b.logits, b.pred, b.ids, b.vals):
                t.zero_()
            g.replay()
        got = b.results()
        for k in ("logits", "pred", "codes", "active_ids", "active_vals"):
            assert np.array_equal(got[k], want[k]), (path, k)
    dm.free()


def test_api_misuse_is_reported_by_error_codes():
    import torch
    from paper_2204_08400_b200 import binding as sl, harness
    dev = torch.device("cuda:0")
    W = [torch.zeros((16, 8), dtype=torch.float32, device=dev), torch.zeros((4, 16), dtype=torch.float32, device=dev)]
    b = [torch.zeros(16, device=dev), torch.zeros(4, device=dev)]
    calib = torch.zeros((10, 8), device=dev)

    def build(**kw):
        args = dict(dims=[8, 16, 4], has_activator=[1, 0], dtype=sl.SLONN_F32, W=W, bias=b, calib_dense=calib, K=2, L=2)
        args.update(kw)
        return sl.slonn_build(**args)

    for kw, code in (
        (dict(dtype=7), "DTYPE"),
        (dict(K=0), "DIM"),
        (dict(K=5, L=4), "DIM"),                                     # K*L = 20 hash nodes > 16 nodes
        (dict(dims=[6, 16, 4]), "ALIGN"),                            # 6 floats = 24 bytes per row: not 16-byte rows
        (dict(calib_dense=None), "ARG"),
        (dict(first_layer_sparse=True), "ARG"),                      # a CSR first layer may not carry an activator
        (dict(hash_nodes_override=[np.array([0, 1, 2, 2]), None]), "ARG"),   # repeated hash node
        (dict(hash_nodes_override=[np.array([0, 1, 2, 99]), None]), "ARG"),  # node id out of range
    ):
        with pytest.raises(sl.SlonnError) as e:
            build(**kw)
        assert e.value.code == sl.ERR[code], (kw, e.value.code)

    wl = custom_workload(64, [32, 64, 8], [1, 0], "f32", n=8, n_cal=80, K=2, L=2, budgets=(2500,))
    dm = harness.DeviceModel(wl)
    batch = harness.DeviceBatch(dm, wl.x, wl.budget_bp)
    with pytest.raises(sl.SlonnError) as e:                          # workspace too small
        sl.slonn_run(dm.model, batch.batch, batch.ws, batch.ws_bytes - 256)
    assert e.value.code == sl.ERR["WORKSPACE"]
    with pytest.raises(sl.SlonnError) as e:                          # misaligned workspace
        sl.slonn_run(dm.model, batch.batch, batch.ws.data_ptr() + 16, batch.ws_bytes)
    assert e.value.code == sl.ERR["WORKSPACE"]
    bad = sl.make_batch(8, batch.bp, None, batch.status, x_dense=batch.x_dense, max_budget_bp=batch.max_bp)   # no logits
    with pytest.raises(sl.SlonnError) as e:
        sl.slonn_run(dm.model, bad, batch.ws, batch.ws_bytes)
    assert e.value.code == sl.ERR["ARG"]
    bad = sl.make_batch(8, batch.bp, batch.logits, batch.status, x_dense=batch.x_dense, max_budget_bp=batch.max_bp,
                        kernel_path=9)
    with pytest.raises(sl.SlonnError) as e:
        sl.slonn_run(dm.model, bad, batch.ws, batch.ws_bytes)
    assert e.value.code == sl.ERR["ARG"]
    batch.run()                                                      # the model is still usable afterwards
    assert batch.results()["status"][0] == 0
    dm.free()


def test_many_tables_and_long_keys():
    # K*L = 96 hash functions, 8 tables of 4096 buckets: most buckets are never reached and fall
    # back to the global ranking
    wl = custom_workload(65, [64, 128, 16], [1, 0], "f32", n=150, n_cal=300, K=12, L=8,
                         budgets=(300, 2500, 10000))
    check(wl)


def test_node_id_width_switches_above_65536_nodes():
    # 65,568 output nodes: the tables hold 32-bit ids (16-bit up to 65,536 nodes)
    from paper_2204_08400_b200 import harness, binding as sl
    wl = custom_workload(66, [32, 64, 65568], [0, 1], "f32", n=6, n_cal=48, K=2, L=2, budgets=(10, 100))
    dm = harness.DeviceModel(wl)
    assert sl.slonn_model_info(dm.model, 1)["id_bytes"] == 4
    dm.free()
    check(wl)
    wl16 = custom_workload(67, [32, 64, 65536], [0, 1], "f32", n=4, n_cal=32, K=2, L=1, budgets=(10,))
    dm = harness.DeviceModel(wl16)
    assert sl.slonn_model_info(dm.model, 1)["id_bytes"] == 2
    dm.free()
    check(wl16)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_budget_split_between_row_and_input_stationary_kernels(dtype):
    # one batch whose budgets lie on both sides of the library's split (35 %), large enough for the
    # library to use the input-stationary kernels by itself: the two launches of a stage must serve
    # disjoint sets of queries and together all of them
    wl = custom_workload(71, [64, 512, 512, 16], [1, 1, 0], dtype, n=640, n_cal=512, K=4, L=2,
                         budgets=(300, 2500, 3500, 3600, 5000, 10000))
    check(wl)


def test_input_stationary_kernel_on_a_wide_list_fed_layer():
    # a 70,000-node budgeted layer fed by the list of the activator layer below: 32-bit ids, a column
    # order over 70,000 nodes, many 64-node passes per query, widths that are no multiple of 32 chunks
    wl = custom_workload(72, [48, 100, 70000], [1, 1], "f32", n=24, n_cal=64, K=3, L=2, budgets=(1000,))
    check(wl)
    # at 50 % the per-query node order no longer fits shared memory: the library must fall back to
    # the row kernel even when the input-stationary one is asked for
    wl = custom_workload(73, [48, 100, 70000], [1, 1], "f32", n=6, n_cal=64, K=3, L=2, budgets=(5000,))
    check(wl)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_input_stationary_kernel_for_a_few_dozen_queries(dtype):
    # too few 64-node warp passes to fill the GPU: one block per (query, 64 nodes) whose warps share the
    # walk over the input list and add their partial sums through shared memory; widths that are no
    # multiple of 64 nodes or 32 chunks, budgets from one node to the whole layer
    wl = custom_workload(76, [40, 296, 200, 12], [1, 1, 0], dtype, n=60, n_cal=200, K=3, L=2,
                         budgets=(30, 500, 2500, 10000))
    check(wl)


@pytest.mark.parametrize("case", [
    dict(seed=5008, dims=[536, 1872, 1712, 806], has_act=[1, 1, 0], n=700, K=7, L=1, budgets=(500, 1500, 9999)),
    dict(seed=5479, dims=[2328, 1568, 1656, 595], has_act=[1, 1, 1], n=37, K=2, L=3, budgets=(10000,)),
])
def test_dynamic_shared_memory_just_below_the_opt_in_limit(case):
    """Layer widths at which a kernel asks for a little less than 48 KB of dynamic shared memory: together with
    its static shared memory that is more than a launch gets without opting in (the four-queries-per-block row
    kernel in the first case, the one-block-per-query input-stationary kernel in the second)."""
    wl = custom_workload(case["seed"], case["dims"], case["has_act"], "bf16", n=case["n"], n_cal=900, K=case["K"],
                         L=case["L"], budgets=case["budgets"])
    check(wl)


def test_widest_layer_input_the_library_accepts():
    """57,600 inputs are 225 KB of staged query, the most a block's shared memory takes; one network without and
    one with an activator on that layer (whose node bitmap sits beside the staged input)."""
    check(custom_workload(75, [57600, 16, 8], [0, 0], "f32", n=6, n_cal=8, K=2, L=1))
    check(custom_workload(76, [57536, 512, 8], [1, 0], "bf16", n=6, n_cal=40, K=3, L=2, budgets=(1000, 10000)))


def test_two_host_threads_run_different_models_at_once():
    """slonn_run may be called from several host threads, each with its own workspace and stream.  The two
    models stage 120 KB and 56 KB of query in the same row kernel, so each thread needs a shared-memory allowance
    the other must not take back between its opt-in and its launch; results must equal the single-threaded ones."""
    import threading
    import torch
    from paper_2204_08400_b200 import harness
    wls = [custom_workload(77, [30000, 64, 16], [1, 0], "f32", n=40, n_cal=60, K=3, L=2, budgets=(1000, 10000)),
           custom_workload(78, [14000, 96, 16], [1, 0], "f32", n=40, n_cal=60, K=3, L=2, budgets=(2500, 10000))]
    dms = [harness.DeviceModel(wl) for wl in wls]
    wants = [harness.run_once(dm, wl.x, wl.budget_bp) for dm, wl in zip(dms, wls)]
    errors = []

    def worker(i):
        try:
            s = torch.cuda.Stream()
            b = harness.DeviceBatch(dms[i], wls[i].x, wls[i].budget_bp)
            for _ in range(40):
                b.logits.fill_(-1)
                with torch.cuda.stream(s):
                    b.run(s)
                s.synchronize()
                got = b.results()
                assert got["status"][0] == 0
                for k in ("logits", "pred", "codes", "active_ids", "active_vals"):
                    assert np.array_equal(got[k], wants[i][k]), k
        except Exception as e:            # reported by the main thread
            errors.append((i, repr(e)))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    for dm in dms:
        dm.free()


def test_input_stationary_kernels_with_an_all_zero_list():
    # biases far below zero: every selected node of the first layer outputs exactly 0, so the next
    # layer's grouped input list is empty and its pre-activations are the biases
    import dataclasses
    wl = custom_workload(74, [32, 96, 64, 8], [1, 1, 0], "bf16", n=300, n_cal=128, K=3, L=2, budgets=(1000, 3000))
    bias = [b.copy() for b in wl.bias]
    bias[0][:] = -1000.0
    wl = dataclasses.replace(wl, bias=bias)
    check(wl)


def test_csr_rows_empty_and_longer_than_one_tile():
    # first layer fed by CSR rows: a query without any nonzero, and rows with 300 nonzeros
    # (more than the 128 the kernel stages at a time)
    import dataclasses
    rng = np.random.default_rng(68)
    base = wl_mod.load("c3", n_queries=8, n_cal=128, budget_bp=1000, dims=[4000, 64, 2000])

    def rows(lengths):
        ids, vals, ip = [], [], [0]
        for n in lengths:
            ids.append(np.sort(rng.choice(4000, n, replace=False)).astype(np.uint32))
            vals.append(np.exp(rng.standard_normal(n)).astype(np.float32))
            ip.append(ip[-1] + n)
        return np.asarray(ip, np.uint64), np.concatenate(ids), np.concatenate(vals)

    wl = dataclasses.replace(base, x=rows([300, 0, 75, 129, 128, 1, 257, 0]), calib=rows([75] * 100 + [300] * 28))
    check(wl)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_zero_inputs_and_tied_logits(dtype):
    # pre-activations of exactly 0 (hash bit 0, ReLU 0) and exactly equal logits (lowest id wins)
    import dataclasses
    wl = custom_workload(69, [64, 96, 16], [1, 0], dtype, n=48, n_cal=200, K=3, L=2, bias_scale=0.0)
    for w in (wl.W_f32[1], wl.W_store[1]):
        w[9] = w[2]; w[13] = w[2]                 # three identical output nodes
    x = wl.x.copy()
    x[::3] = 0.0                                  # every third query is all zeros
    wl = dataclasses.replace(wl, x=x)
    check(wl)


# ---- hash nodes always active and absent from the lists (Sec. 3.4 variant) ---------

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_free_hash_nodes_small_mlp(dtype):
    wl = custom_workload(90, [136, 200, 96, 24], [1, 1, 0], dtype, n=300, n_cal=700, K=4, L=2,
                         budgets=(100, 1000, 2500, 5000, 9300, 10000))   # 9300: B above the 88 non-hash nodes of layer 2
    wl.free_hash_nodes = True
    check(wl)


def test_free_hash_nodes_output_activator_three_tables_and_list_cap():
    wl = custom_workload(91, [72, 160, 328], [1, 1], "f32", n=120, n_cal=500, K=3, L=3, list_cap=120,
                         budgets=(100, 700, 3300, 10000))
    wl.free_hash_nodes = True
    check(wl)


def test_free_hash_nodes_c2_reduced():
    for bp in (500, 2500, 10000):
        wl = wl_mod.load("c2", n_queries=600, n_cal=2048, budget_bp=bp, free_hash_nodes=True)
        check(wl, expect_build=(bp == 500))


def test_free_hash_nodes_c4_reduced_and_serialization_round_trip():
    from paper_2204_08400_b200 import binding as sl, harness
    wl = wl_mod.load("c4", n_queries=3, n_cal=512, budget_bp=1000, dims=[512, 1024, 1024, 1024, 1024, 1024, 1024, 1024, 1024, 200],
                     free_hash_nodes=True)
    check(wl)
    dm = harness.DeviceModel(wl, n_cal=512)
    want = harness.run_once(dm, wl.x, wl.budget_bp)
    blob = sl.slonn_serialize(dm.model)
    built, dm.model = dm.model, sl.slonn_deserialize(blob, dm.W, dm.bias)
    assert dm.model.free_hash_nodes
    got = harness.run_once(dm, wl.x, wl.budget_bp)
    for k in ("logits", "pred", "codes", "active_indptr", "active_ids", "active_vals"):
        assert np.array_equal(got[k], want[k]), k
    sl.slonn_free(built)
    dm.free()
