"""The benchmark's algorithmic byte counts (what roofline.achieved divides by time), checked by hand on a
toy network: row kernels count whole weight rows, the input-stationary kernels count selected nodes x
input list entries, and the split between the two follows the library's rule."""
import os
import sys
import types

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def toy(dtype="bf16", n=16000):     # enough queries for 64-node warp passes to fill the GPU in every layer
    wl = types.SimpleNamespace(dims=[64, 200, 200, 10], has_act=[1, 1, 0], dtype=dtype, first_sparse=False, K=10, L=2)
    return wl, np.full(n, 1000, np.uint16)


def test_budget_nodes_rounds_half_up_with_a_floor_of_one():
    bp = np.array([1, 25, 1000, 10000], np.uint16)
    assert bench.budget_nodes(bp, 200).tolist() == [1, 1, 20, 200]     # 0.02 -> 1, 0.5 -> 1, 20, 200
    assert bench.budget_nodes(np.array([250], np.uint16), 10).tolist() == [1]   # 0.25 -> floor of one node


def test_row_and_input_stationary_bytes_of_a_toy_network():
    wl, bp = toy()
    n, esz, H = bp.size, 2, 20
    rows, cols, layer, grouped = bench.gathered_bytes(wl, bp)
    # layer 0: dense input, 20 selected rows of 64 weights
    assert rows == n * 20 * 64 * esz
    # layer 1: fed by layer 0's 20-entry list, own activator: (20 selected + 20 hash nodes) x 20 entries
    assert layer == n * (20 + H) * 20 * esz
    # layer 2: fed by layer 1's 20-entry list, every one of its 10 nodes
    assert cols == n * 10 * 20 * esz


def test_forced_rows_count_whole_rows_everywhere():
    wl, bp = toy("f32")
    n, esz = bp.size, 4
    rows, cols, layer, grouped = bench.gathered_bytes(wl, bp, force_rows=True)
    assert (cols, layer) == (0, 0)
    assert rows == n * (20 * 64 + 20 * 200 + 10 * 200) * esz


def test_budgets_above_the_split_take_the_row_kernels():
    wl, _ = toy()
    bp = np.array([1000] * 12000 + [5000] * 4000, np.uint16)
    rows, cols, layer, grouped = bench.gathered_bytes(wl, bp)
    esz, H = 2, 20
    low, high = 12000, 4000
    assert layer == low * (20 + H) * 20 * esz
    assert cols == low * 10 * 20 * esz
    assert rows == (low * 20 + high * 100) * 64 * esz + high * 100 * 200 * esz + high * 10 * 200 * esz


def test_small_batches_keep_the_row_kernels():
    wl, bp = toy(n=40)      # 40 queries x 20 nodes: far too few warp passes, and the layers are narrow
    rows, cols, layer, grouped = bench.gathered_bytes(wl, bp)
    assert (cols, layer) == (0, 0)
    assert rows == 40 * (20 * 64 + 20 * 200 + 10 * 200) * 2


def test_empty_batch_has_no_bytes():
    wl, _ = toy()
    assert bench.gathered_bytes(wl, np.zeros(0, np.uint16)) == (0, 0, 0, 0)


def test_row_queries_of_a_layer_without_activator_are_counted_as_grouped():
    wl = types.SimpleNamespace(dims=[64, 2048, 1024], has_act=[1, 0], dtype="bf16", first_sparse=False, K=10, L=2)
    bp = np.full(16000, 5000, np.uint16)        # above the split: row kernels; the second layer computes every node
    rows, cols, layer, grouped = bench.gathered_bytes(wl, bp)
    assert (cols, layer) == (0, 0)
    assert rows == 16000 * 1024 * 64 * 2        # first layer: 1024 selected rows of 64 weights
    assert grouped == 16000 * 1024 * 2048 * 2   # second layer: every row, whole, per query
