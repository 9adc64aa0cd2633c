"""Pins for the oracle's free-hash-node variant (Sec. 3.4: a hash function's dot product is the
pre-activation of a real node, so that node's output comes with the key).  In this variant a
layer's K*L hash nodes are always active and its ranked lists hold the other nodes only; the
budget counts list nodes.  CPU only."""
import numpy as np
import pytest

from oracle import oracle as orc
from test_oracle_method import closed_form_active, relu_inputs
from test_oracle_pins import dense_forward64, tiny_model


def make_pair(rng, dims, has_act, K, L, list_cap=0, seed=5, n_cal=300):
    """The same network trained on the same rows with the same hash nodes, in both modes."""
    W = [rng.standard_normal((dims[l + 1], dims[l])).astype(np.float32) / np.float32(np.sqrt(dims[l]))
         for l in range(len(dims) - 1)]
    b = [(rng.standard_normal(dims[l + 1]) * 0.3).astype(np.float32) for l in range(len(dims) - 1)]
    plain = orc.OracleModel(dims, has_act, W, b, V=4, K=K, L=L, list_cap=0)
    free = orc.OracleModel(dims, has_act, W, b, V=4, K=K, L=L, list_cap=list_cap, free_hash_nodes=True)
    calib = relu_inputs(rng, n_cal, dims[0])
    plain.build(calib_dense=calib, seed=seed)
    free.build(calib_dense=calib, seed=seed)
    return plain, free


def test_lists_are_the_plain_rankings_with_the_hash_nodes_deleted():
    # Leaving a node out of a ranking does not reorder the others.  Layer 0 sees the same
    # calibration activations in both modes (training uses complete activations), and so does
    # every later layer.
    rng = np.random.default_rng(70)
    plain, free = make_pair(rng, [20, 48, 40, 6], [1, 1, 0], K=3, L=2)
    for l in (0, 1):
        hn = plain.hash_nodes(l)
        assert np.array_equal(hn, free.hash_nodes(l))
        N = plain.dims[l + 1]
        assert free.cap(l) == N - hn.size
        rp, rf = plain.rank(l), free.rank(l)
        for b in range(2):
            for key in range(8):
                keep = rp[b, key][~np.isin(rp[b, key], hn)]
                assert np.array_equal(rf[b, key], keep)


def test_list_cap_keeps_the_first_entries_of_the_filtered_ranking():
    rng = np.random.default_rng(71)
    _, full = make_pair(rng, [16, 40, 5], [1, 0], K=2, L=2)
    rng = np.random.default_rng(71)
    _, capped = make_pair(rng, [16, 40, 5], [1, 0], K=2, L=2, list_cap=9)
    assert capped.cap(0) == 9
    assert np.array_equal(capped.rank(0), full.rank(0)[:, :, :9])


@pytest.mark.parametrize("L", [1, 2, 3])
def test_active_set_is_hash_nodes_plus_closed_form_selection(L):
    rng = np.random.default_rng(72 + L)
    D, N, K = 12, 41, 2
    H = K * L
    W = [rng.standard_normal((N, D)).astype(np.float32), rng.standard_normal((4, N)).astype(np.float32)]
    b = [rng.standard_normal(N).astype(np.float32), np.zeros(4, np.float32)]
    m = orc.OracleModel([D, N, 4], [1, 0], W, b, V=4, K=K, L=L, free_hash_nodes=True)
    hn = rng.choice(N, H, replace=False).astype(np.uint32)
    others = np.setdiff1d(np.arange(N, dtype=np.uint32), hn)
    tabs = np.stack([np.stack([rng.permutation(others) for _ in range(1 << K)]) for _ in range(L)]).astype(np.uint32)
    m.set_tables(0, hn, tabs)
    x = rng.standard_normal((20, D)).astype(np.float32)
    prev = None
    for bp in (100, 1000, 2500, 5000, 8000, 9000, 10000):
        r = m.run(np.full(20, bp, np.uint16), x_dense=x)
        B = orc.budget_nodes(bp, N)
        take = min(B, N - H)
        ip = r["active_indptr"].astype(np.int64)
        assert ip[-1] == 20 * (take + H)
        sets = []
        for q in range(20):
            ids = r["active_ids"][ip[q]:ip[q + 1]]
            assert ids.size == take + H
            assert np.all(np.diff(ids.astype(np.int64)) > 0)
            # closed form on the lists (ids relabelled to 0..N-H-1 for the helper, then mapped back)
            pos = {int(n): i for i, n in enumerate(others)}
            lists = [np.array([pos[int(n)] for n in tabs[t, r["codes"][q, 0, t]]]) for t in range(L)]
            chosen = others[closed_form_active(lists, take)] if take else np.array([], np.uint32)
            assert np.array_equal(ids, np.sort(np.concatenate([hn, chosen])))
            sets.append(set(ids.tolist()))
        if prev is not None:
            for q in range(20):
                assert prev[q] <= sets[q]
        prev = sets


def test_values_are_those_of_the_plain_model_on_the_same_set():
    # An active node's value depends only on the layer input: with one activator layer the
    # free variant's hidden values must equal the dense layer's values at the active ids, hash
    # nodes included (their sign is the key bit).
    rng = np.random.default_rng(76)
    _, free = make_pair(rng, [24, 64, 7], [1, 0], K=3, L=2)
    x = relu_inputs(rng, 30, 24)
    r = free.run(np.full(30, 2000, np.uint16), x_dense=x, mode=orc.REF64)
    hidden = np.maximum(x.astype(np.float64) @ free.W[0].astype(np.float64).T + free.bias[0], 0.0)
    ip = r["active_indptr"].astype(np.int64)
    hn = free.hash_nodes(0)
    for q in range(30):
        ids = r["active_ids"][ip[q]:ip[q + 1]]
        vals = r["active_vals"][ip[q]:ip[q + 1]]
        assert np.allclose(vals, hidden[q, ids], rtol=1e-12, atol=1e-12)
        assert set(hn.ravel().tolist()) <= set(ids.tolist())
        for t in range(2):
            for j in range(3):
                assert bool((r["codes"][q, 0, t] >> j) & 1) == bool(hidden[q, hn[t, j]] > 0)
        # the logits use exactly these values and zeros elsewhere
        h = np.zeros(64); h[ids] = vals
        want = h @ free.W[1].astype(np.float64).T + free.bias[1]
        assert np.allclose(r["logits"][q], want, rtol=1e-12, atol=1e-12)


def test_full_budget_is_the_dense_network_in_both_modes():
    rng = np.random.default_rng(77)
    plain, free = make_pair(rng, [32, 48, 40, 7], [1, 1, 0], K=3, L=2)
    x = relu_inputs(rng, 11, 32)
    bp = np.full(11, 10000, np.uint16)
    a = plain.run(bp, x_dense=x)
    b = free.run(bp, x_dense=x)
    assert np.array_equal(a["logits"], b["logits"]) and np.array_equal(a["active_ids"], b["active_ids"])
    want = dense_forward64(free, x)
    c = free.run(bp, x_dense=x, mode=orc.REF64)
    assert np.max(np.abs(c["logits"] - want)) <= 1e-12 * np.max(np.abs(want))


def test_budget_above_the_non_hash_nodes_takes_every_node():
    rng = np.random.default_rng(78)
    _, free = make_pair(rng, [16, 20, 4], [1, 0], K=3, L=2)   # 6 hash nodes of 20
    x = relu_inputs(rng, 5, 16)
    for bp, count in ((6500, 13 + 6), (7000, 20), (9900, 20)):  # round(0.65*20)=13 < 14; 14 = N - H
        r = free.run(np.full(5, bp, np.uint16), x_dense=x)
        assert r["active_indptr"][-1] == 5 * count
