"""The benchmark's byte counts (what roofline.achieved divides by time), checked by hand on toy networks.
The counts are driven by launch records as the library's traced run returns them; here the records are
written out by hand, so no GPU is needed."""
import numpy as np

from paper_2204_08400_b200 import accounting as acc


def toy(esz=2):
    return acc.NetShape(dims=[64, 200, 200, 10], has_act=[1, 1, 0], esz=esz, K=10, L=2)


def rec(stage, layer, lo=0, hi=10000, skips_full=False, cols_bp=0, ms=1.0):
    return dict(stage=stage, layer=layer, bp_lo=lo, bp_hi=hi, skips_full=skips_full, cols_bp=cols_bp, ms=ms)


def test_node_count_rounds_half_up_with_a_floor_of_one():
    bp = np.array([1, 25, 1000, 10000])
    assert acc.layer_nodes(bp, 200).tolist() == [1, 1, 20, 200]       # 0.02 -> 1, 0.5 -> 1, 20, 200
    assert acc.layer_nodes(np.array([250]), 10).tolist() == [1]       # 0.25 -> floor of one node
    assert acc.layer_nodes(np.array([1000, 9900]), 200, pre=20).tolist() == [40, 200]   # always-on hash nodes


def test_first_layer_rows_and_hash_rows_are_whole_rows_in_every_count():
    sh, n = toy(), 1000
    bp = np.full(n, 1000)                     # 20 of 200 nodes
    sel = acc.launch_bytes(sh, rec("hash_select", 0), bp)
    want = n * (20 * 64 * 2 + 2 * 20 * 2)     # 20 hash rows of 64 bf16 weights + two lists of 20 two-byte ids
    assert sel["as_run"] == sel["algorithmic"] == sel["row_granular"] == want
    rows = acc.launch_bytes(sh, rec("gather_dot", 0), bp)
    assert rows["as_run"] == rows["algorithmic"] == rows["row_granular"] == n * 20 * 64 * 2


def test_list_fed_layer_row_form_against_input_stationary_form():
    sh, n = toy(), 1000
    bp = np.full(n, 1000)
    # layer 1 is fed by layer 0's 20-entry list and selects 20 nodes
    r = acc.launch_bytes(sh, rec("gather_dot", 1), bp)
    assert r["as_run"] == r["row_granular"] == n * 20 * 200 * 2
    assert r["algorithmic"] == n * 20 * 20 * 2
    c = acc.launch_bytes(sh, rec("gather_cols", 1), bp)
    assert c["as_run"] == c["algorithmic"] == n * 20 * 20 * 2 and c["row_granular"] == n * 20 * 200 * 2
    whole = acc.launch_bytes(sh, rec("layer_cols", 1), bp)       # hash functions, lists and nodes in one launch
    assert whole["as_run"] == whole["algorithmic"] == n * ((20 + 20) * 20 * 2 + 2 * 20 * 2)
    # the output layer computes every one of its 10 nodes from layer 1's list
    o = acc.launch_bytes(sh, rec("gather_cols", 2), bp)
    assert o["as_run"] == n * 10 * 20 * 2 and o["row_granular"] == n * 10 * 200 * 2


def test_budget_ranges_and_skipped_full_budget_queries():
    sh = toy()
    bp = np.array([1000] * 6 + [5000] * 3 + [10000] * 2)
    low = acc.launch_bytes(sh, rec("gather_cols", 1, 0, 3500), bp)
    assert low["queries"] == 6 and low["as_run"] == 6 * 20 * 20 * 2
    high = acc.launch_bytes(sh, rec("gather_dot", 1, 3501, 10000, skips_full=True), bp)
    assert high["queries"] == 3 and high["as_run"] == 3 * 100 * 200 * 2 and high["algorithmic"] == 3 * 100 * 100 * 2
    full = acc.launch_bytes(sh, rec("full_rows", 1, 10000, 10000), bp)
    assert full["queries"] == 2 and full["as_run"] == full["algorithmic"] == 2 * 200 * 200 * 2
    assert acc.launch_bytes(sh, rec("gather_dot", 1, 20000, 30000), bp)["queries"] == 0
    # four queries per block: the same row-wise count as the one-query row kernel for the queries it serves
    grouped = acc.launch_bytes(sh, rec("group_rows", 1, 2001, 10000, skips_full=True), bp)
    assert grouped["queries"] == 3 and grouped["as_run"] == high["as_run"] and grouped["algorithmic"] == high["algorithmic"]
    assert acc.kernel_name(sh, rec("group_rows", 1)) == "group_rows_kernel"


def test_whole_network_launch_takes_each_layers_form_from_the_record():
    # the worked count of the 784-1024-1024-10 bf16 network at a 10 % budget (102 nodes per hidden layer):
    # 20 hash rows and 102 rows of 784 weights, then 20 hash functions and 102 nodes over the 102-entry list,
    # then 10 output nodes over the 102-entry list, plus two lists of 102 two-byte ids per hidden layer
    sh = acc.NetShape(dims=[784, 1024, 1024, 10], has_act=[1, 1, 0], esz=2, K=10, L=2)
    bp = np.array([1000])
    alg = 31360 + 102 * 1568 + 40 * 102 + 2 * 102 * 102 + 20 * 102 + 8 * 102
    assert alg == 219040
    cols = acc.launch_bytes(sh, rec("fused", None, cols_bp=1250), bp)
    assert cols["algorithmic"] == alg
    # as run: the second layer input-stationary, the output layer's 10 rows whole
    assert cols["as_run"] == alg - 20 * 102 + 10 * 1024 * 2
    rows = acc.launch_bytes(sh, rec("fused", None, cols_bp=0), bp)
    assert rows["algorithmic"] == alg
    assert rows["as_run"] == rows["row_granular"] == 31360 + 102 * 1568 + (20 + 102 + 10) * 2048 + 8 * 102
    assert acc.step_bytes(sh, bp) == dict(algorithmic=alg, row_granular=rows["row_granular"])


def test_csr_first_layer_and_tensor_core_records():
    sh = acc.NetShape(dims=[1000, 128, 500], has_act=[0, 1], esz=4, K=10, L=2, first_sparse=True)
    bp = np.array([1000, 1000, 1000])
    first = acc.launch_bytes(sh, rec("sparse_first", 0), bp, x_nnz=np.array([75, 0, 5]))
    assert first["as_run"] == first["algorithmic"] == 80 * 128 * 4
    out = acc.launch_bytes(sh, rec("gather_dot", 1), bp)          # dense 128-wide input, 50 of 500 nodes
    assert out["as_run"] == out["algorithmic"] == 3 * 50 * 128 * 4
    tc = acc.launch_bytes(toy(), rec("dense_tc", None, 10000, 10000), np.array([10000, 500, 10000]))
    assert tc["queries"] == 2 and tc["flops"] == 2 * 2.0 * (64 * 200 + 200 * 200 + 200 * 10) and tc["as_run"] == 0


def test_records_group_by_kernel_and_short_rows_name_their_kernel():
    sh = acc.NetShape(dims=[1000, 128, 500], has_act=[0, 1], esz=4, K=10, L=2, first_sparse=True)
    bp = np.full(4, 1000)
    recs = [rec("sparse_first", 0, ms=0.5), rec("hash_select", 1, ms=0.25), rec("gather_dot", 1, ms=1.5), rec("argmax", None, ms=0.1)]
    k = acc.per_kernel(sh, recs, bp, x_nnz=np.full(4, 10))
    assert set(k) == {"sparse_first_layer_kernel", "hash_select_kernel", "gather_short_kernel", "argmax_kernel"}
    assert k["gather_short_kernel"]["launches"] == 1 and k["gather_short_kernel"]["ms"] == 1.5
    assert k["gather_short_kernel"]["algorithmic"] == 4 * 50 * 128 * 4
    assert k["argmax_kernel"]["algorithmic"] == 0


def test_empty_batch_has_no_bytes():
    assert acc.launch_bytes(toy(), rec("fused", None), np.zeros(0, np.int64))["as_run"] == 0
