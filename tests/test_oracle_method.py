"""Pins for the oracle's Node-Activator training (Algorithm 1, FreeHash
sampling of Sec. 3.4) and the SLO-aware forward pass (Fig. 2, Sec. 3.3):
brute force on tiny layers, closed forms and invariants.  CPU only."""
from collections import defaultdict

import numpy as np
import pytest

from oracle import oracle as orc
from test_oracle_pins import tiny_model


def relu_inputs(rng, n, D):
    return np.maximum(rng.standard_normal((n, D)), 0).astype(np.float32)


# ---------------------------------------------------------------------------
# Selection rule (Fig. 2 step 4: the top k% of the sorted list)
# ---------------------------------------------------------------------------

def closed_form_active(lists, B):
    """B nodes with the smallest priority p(n) = min_b(rank_b(n) * L + b)."""
    L = len(lists)
    N = len(lists[0])
    prio = np.full(N, np.iinfo(np.int64).max, dtype=np.int64)
    for b, lst in enumerate(lists):
        for r, n in enumerate(lst):
            prio[n] = min(prio[n], r * L + b)
    order = sorted(range(N), key=lambda n: prio[n])
    return np.sort(np.array(order[:B], dtype=np.uint32))


def hand_tables(rng, N, K, L):
    return np.stack([np.stack([rng.permutation(N) for _ in range(1 << K)]) for _ in range(L)]).astype(np.uint32)


@pytest.mark.parametrize("L", [1, 2, 3])
def test_selection_matches_closed_form_and_nests(L):
    rng = np.random.default_rng(20 + L)
    D, N, K = 12, 37, 2
    m = tiny_model(rng, [D, N, 4], [1, 0], K=K, L=L)
    hn = rng.choice(N, K * L, replace=False).astype(np.uint32)
    tabs = hand_tables(rng, N, K, L)
    m.set_tables(0, hn, tabs)
    x = rng.standard_normal((25, D)).astype(np.float32)
    prev = None
    for bp in (300, 1000, 2500, 5000, 7500, 9000, 10000):
        r = m.run(np.full(25, bp, np.uint16), x_dense=x)
        B = orc.budget_nodes(bp, N)
        ip = r["active_indptr"].astype(np.int64)
        sets = []
        for q in range(25):
            ids = r["active_ids"][ip[q]:ip[q + 1]]
            assert ids.size == B                                  # |active| = B
            assert np.all(np.diff(ids.astype(np.int64)) > 0)      # strictly ascending, distinct
            assert ids.max() < N
            lists = [tabs[b, r["codes"][q, 0, b]] for b in range(L)]
            assert np.array_equal(ids, closed_form_active(lists, B))
            if L == 1:                                            # literally the list prefix
                assert np.array_equal(ids, np.sort(lists[0][:B]))
            sets.append(set(ids.tolist()))
        if prev is not None:                                      # monotone nesting in the budget
            for q in range(25):
                assert prev[q] <= sets[q]
        prev = sets


def test_identical_inputs_collide_and_small_perturbations_mostly_do():
    # LSH property (Sec. 3.1): collision probability grows with similarity
    rng = np.random.default_rng(24)
    m = tiny_model(rng, [64, 128, 8], [1, 0], K=6, L=2)
    calib = relu_inputs(rng, 300, 64)
    m.build(calib_dense=calib, seed=1)
    x = relu_inputs(rng, 200, 64)
    bp = np.full(200, 2500, np.uint16)
    a = m.run(bp, x_dense=x)["codes"]
    b = m.run(bp, x_dense=x.copy())["codes"]
    assert np.array_equal(a, b)
    near = m.run(bp, x_dense=(x * np.float32(1.0 + 1e-4)))["codes"]
    far = m.run(bp, x_dense=relu_inputs(rng, 200, 64))["codes"]
    same_near = np.mean(np.all(a == near, axis=(1, 2)))
    same_far = np.mean(np.all(a == far, axis=(1, 2)))
    assert same_near > 0.9 and same_near > same_far


# ---------------------------------------------------------------------------
# Algorithm 1 by brute force on tiny layers
# ---------------------------------------------------------------------------

def brute_force_tables(m, l, inputs_l, hash_nodes, K, L):
    """Algorithm 1 with a dict of lists; float64 everywhere except the layer
    activations, which are taken as given (float32 values)."""
    N = m.dims[l + 1]
    last = (l == m.n_layers - 1)
    acts = []
    for x in inputs_l:
        z = np.array([orc.dot_canon32(m.W[l][n], x, m.V, m.bias[l][n]) for n in range(N)], dtype=np.float32)
        acts.append(z if last else np.where(z > 0, z, np.float32(0)))
    acts = np.array(acts, dtype=np.float32)
    members = [defaultdict(list) for _ in range(L)]
    for s, a in enumerate(acts):
        for b in range(L):
            key = sum((1 << j) for j in range(K) if a[hash_nodes[b][j]] > 0)
            members[b][key].append(s)
    glob = np.zeros(N)
    for a in acts:
        glob = glob + a.astype(np.float64)
    def ranking(score):
        return sorted(range(N), key=lambda n: (-score[n], n))
    out = np.zeros((L, 1 << K, N), dtype=np.uint32)
    for b in range(L):
        for key in range(1 << K):
            if members[b][key]:
                sc = np.zeros(N)
                for s in members[b][key]:
                    sc = sc + acts[s].astype(np.float64)
                out[b, key] = ranking(sc)
            else:
                out[b, key] = ranking(glob)
    return out, acts


def test_algorithm1_brute_force_two_layers():
    rng = np.random.default_rng(30)
    K, L = 3, 2
    m = tiny_model(rng, [10, 16, 12, 4], [1, 1, 0], K=K, L=L)
    calib = relu_inputs(rng, 64, 10)
    m.build(calib_dense=calib, seed=77, keep_scores=True)
    hn0, hn1 = m.hash_nodes(0), m.hash_nodes(1)
    want0, acts0 = brute_force_tables(m, 0, calib, hn0, K, L)
    assert np.array_equal(m.rank(0), want0)
    # layer 2 is trained on the complete activations of layer 1 (Sec. 4.1)
    want1, _ = brute_force_tables(m, 1, acts0, hn1, K, L)
    assert np.array_equal(m.rank(1), want1)


def test_algorithm1_budgeted_output_layer_uses_raw_scores():
    rng = np.random.default_rng(31)
    K, L = 2, 2
    m = tiny_model(rng, [9, 6, 14], [0, 1], K=K, L=L)
    calib = relu_inputs(rng, 40, 9)
    m.build(calib_dense=calib, seed=5)
    # hidden layer has no activator: its complete ReLU activations feed the output layer
    h = np.array([[max(orc.dot_canon32(m.W[0][n], x, 4, m.bias[0][n]), 0.0) for n in range(6)] for x in calib],
                 dtype=np.float32)
    want, _ = brute_force_tables(m, 1, h, m.hash_nodes(1), K, L)
    assert np.array_equal(m.rank(1), want)


def test_build_invariants():
    rng = np.random.default_rng(32)
    K, L, N = 4, 2, 50
    m = tiny_model(rng, [20, N, 6], [1, 0], K=K, L=L)
    calib = relu_inputs(rng, 500, 20)
    m.build(calib_dense=calib, seed=9, keep_scores=True)
    rank, score, cnt = m.rank(0), m.score(0), m.bucket_count(0)
    acts = np.array([[max(orc.dot_canon32(m.W[0][n], x, 4, m.bias[0][n]), 0.0) for n in range(N)] for x in calib])
    assert np.array_equal(cnt.sum(axis=1), np.full(L, 500))          # every sample lands in one bucket per table
    for b in range(L):
        # the buckets partition the samples: bucket sums add up to the column sums
        assert np.allclose(score[b].sum(axis=0), acts.sum(axis=0), rtol=1e-12, atol=1e-9)
        for key in range(1 << K):
            assert np.array_equal(np.sort(rank[b, key]), np.arange(N))   # a permutation of the layer
            if cnt[b, key]:
                s = score[b, key][rank[b, key]]
                assert np.all(np.diff(s) <= 0)                        # highest to lowest
                ties = np.diff(s) == 0
                assert np.all(np.diff(rank[b, key].astype(np.int64))[ties] > 0)
    hn = m.hash_nodes(0).reshape(-1)
    assert len(set(hn.tolist())) == K * L


def test_list_cap_truncates_lists_and_keeps_results():
    rng = np.random.default_rng(33)
    dims = [16, 40, 5]
    full = tiny_model(rng, dims, [1, 0], K=3, L=2)
    capped = orc.OracleModel(dims, [1, 0], full.W, full.bias, V=4, K=3, L=2, list_cap=12)
    calib = relu_inputs(rng, 120, 16)
    full.build(calib_dense=calib, seed=4)
    capped.build(calib_dense=calib, seed=4)
    assert np.array_equal(capped.rank(0), full.rank(0)[:, :, :12])
    x = relu_inputs(rng, 9, 16)
    for bp in (1000, 2500, 3000, 10000):   # B = 4, 10, 12, 40 (all nodes)
        a = full.run(np.full(9, bp, np.uint16), x_dense=x)
        b = capped.run(np.full(9, bp, np.uint16), x_dense=x)
        assert np.array_equal(a["active_ids"], b["active_ids"])
        assert np.array_equal(a["logits"], b["logits"])
    with pytest.raises(RuntimeError):
        capped.run(np.full(9, 5000, np.uint16), x_dense=x)   # B = 20 > cap


# ---------------------------------------------------------------------------
# FreeHash sampling (Sec. 3.4): probability proportional to activation variance
# ---------------------------------------------------------------------------

def test_sampling_never_draws_zero_variance_while_positive_remain():
    var = np.array([0, 3.0, 0, 1.0, 0, 0, 2.0, 0.5, 0, 0])
    for seed in range(200):
        out = orc.sample_hash_nodes(var, 4, seed, 0)
        assert set(out.tolist()) == {1, 3, 6, 7}
        out6 = orc.sample_hash_nodes(var, 6, seed, 0)
        assert len(set(out6.tolist())) == 6 and set(out6[:4].tolist()) == {1, 3, 6, 7}


def test_sampling_first_draw_frequencies_follow_variance():
    var = np.array([1.0, 2.0, 3.0, 4.0, 0.0, 10.0])
    counts = np.zeros(6)
    n = 20000
    for seed in range(n):
        counts[orc.sample_hash_nodes(var, 2, seed, 1)[0]] += 1
    expect = var / var.sum() * n
    assert counts[4] == 0
    nz = expect > 0
    chi2 = np.sum((counts[nz] - expect[nz]) ** 2 / expect[nz])
    assert chi2 < 30.0          # 4 degrees of freedom; 30 is far in the tail


def test_sampling_uses_population_variance_of_activations():
    rng = np.random.default_rng(35)
    m = tiny_model(rng, [8, 12, 3], [1, 0], K=2, L=2)
    calib = relu_inputs(rng, 90, 8)
    m.build(calib_dense=calib, seed=2)
    acts = np.array([[max(orc.dot_canon32(m.W[0][n], x, 4, m.bias[0][n]), 0.0) for n in range(12)] for x in calib])
    assert np.allclose(m.var(0), acts.var(axis=0), rtol=1e-12, atol=1e-15)
    assert np.array_equal(m.hash_nodes(0).reshape(-1), orc.sample_hash_nodes(m.var(0), 4, 2, 0))


# ---------------------------------------------------------------------------
# Forward pass by brute force (float64), and its invariants
# ---------------------------------------------------------------------------

def brute_force_forward64(m, x, bp):
    """k% forward propagation written out with numpy float64 and Python loops."""
    a = x.astype(np.float64)
    codes, sets = [], []
    for l in range(m.n_layers):
        W = m.W[l].astype(np.float64); b = m.bias[l].astype(np.float64)
        N = m.dims[l + 1]
        last = l == m.n_layers - 1
        if m.has_act[l]:
            hn, rank = m.hash_nodes(l), m.rank(l)
            keys = []
            for t in range(m.L):
                key = 0
                for j in range(m.K):
                    if float(W[hn[t, j]] @ a + b[hn[t, j]]) > 0:
                        key |= 1 << j
                keys.append(key)
            B = max(1, (int(bp) * N + 5000) // 10000)
            chosen = []
            r = 0
            while len(chosen) < B:
                for t in range(m.L):
                    n = int(rank[t, keys[t], r])
                    if n not in chosen and len(chosen) < B:
                        chosen.append(n)
                r += 1
            chosen = sorted(chosen)
            codes.append(keys); sets.append(chosen)
        else:
            chosen = list(range(N))
        out = np.zeros(N)
        for n in chosen:
            z = float(W[n] @ a + b[n])
            out[n] = z if last else max(z, 0.0)
        a = out
    return a, codes, sets


def test_forward_pass_brute_force_ref64():
    rng = np.random.default_rng(40)
    m = tiny_model(rng, [14, 20, 18, 6], [1, 1, 0], K=3, L=2)
    m.build(calib_dense=relu_inputs(rng, 150, 14), seed=8)
    x = relu_inputs(rng, 30, 14)
    bps = rng.choice([500, 1000, 2500, 5000, 10000], 30).astype(np.uint16)
    r = m.run(bps, x_dense=x, mode=orc.REF64)
    ip = r["active_indptr"].astype(np.int64)
    for q in range(30):
        logits, codes, sets = brute_force_forward64(m, x[q], bps[q])
        assert np.array_equal(r["codes"][q], np.array(codes, dtype=np.uint16))
        for a in range(2):
            assert r["active_ids"][ip[2 * q + a]:ip[2 * q + a + 1]].tolist() == sets[a]
        assert np.allclose(r["logits"][q], logits, rtol=1e-12, atol=1e-14)
        assert r["pred"][q] == int(np.argmax(logits))


def test_active_hash_nodes_agree_with_their_bits():
    # FreeHash (Def. 2): a hash bit is the sign of a real node of the same layer,
    # so whenever that node is computed its value is positive iff the bit is set
    rng = np.random.default_rng(41)
    m = tiny_model(rng, [30, 64, 48, 5], [1, 1, 0], K=4, L=2)
    m.build(calib_dense=relu_inputs(rng, 400, 30), seed=12)
    x = relu_inputs(rng, 60, 30)
    r = m.run(np.full(60, 5000, np.uint16), x_dense=x)
    ip = r["active_indptr"].astype(np.int64)
    checked = 0
    for q in range(60):
        for a in range(2):
            ids = r["active_ids"][ip[2 * q + a]:ip[2 * q + a + 1]]
            vals = r["active_vals"][ip[2 * q + a]:ip[2 * q + a + 1]]
            hn = m.hash_nodes(a)
            for t in range(m.L):
                for j in range(m.K):
                    pos = np.searchsorted(ids, hn[t, j])
                    if pos < ids.size and ids[pos] == hn[t, j]:
                        assert (vals[pos] > 0) == bool((r["codes"][q, a, t] >> j) & 1)
                        checked += 1
    assert checked > 100


def test_sparse_operand_first_layer_and_budgeted_output():
    # extreme-classification shape: sparse features -> small hidden layer -> wide
    # output layer carrying the only Node Activator (Sec. 4, model paragraph)
    rng = np.random.default_rng(42)
    D, Hd, N = 500, 16, 300
    m = tiny_model(rng, [D, Hd, N], [0, 1], K=4, L=2, first_sparse=True)

    def csr(n, nnz):
        ids = np.stack([np.sort(rng.choice(D, nnz, replace=False)) for _ in range(n)]).astype(np.uint32)
        vals = np.exp(rng.standard_normal((n, nnz))).astype(np.float32)
        return np.arange(n + 1, dtype=np.uint64) * np.uint64(nnz), ids.reshape(-1), vals.reshape(-1)

    m.build(calib_csr=csr(200, 40), seed=3)
    xs = csr(20, 40)
    bp = np.full(20, 1000, np.uint16)
    r32 = m.run(bp, x_csr=xs, mode=orc.CANON32)
    r64 = m.run(bp, x_csr=xs, mode=orc.REF64)
    assert r32["logits"].shape == (20, 30) and r32["logit_ids"].shape == (20, 30)
    same = np.all(r32["codes"] == r64["codes"], axis=(1, 2))
    assert same.mean() > 0.9
    for q in np.nonzero(same)[0]:
        assert np.array_equal(r32["logit_ids"][q], r64["logit_ids"][q])
        rel = np.max(np.abs(r32["logits"][q] - r64["logits"][q])) / np.max(np.abs(r64["logits"][q]))
        assert rel < 1e-5
    # hidden layer against a float64 scatter + matrix product
    dense = np.zeros((20, D))
    ids = xs[1].reshape(20, 40); vals = xs[2].reshape(20, 40)
    for q in range(20):
        dense[q, ids[q]] = vals[q]
    h = np.maximum(dense @ m.W[0].astype(np.float64).T + m.bias[0], 0)
    for q in np.nonzero(same)[0]:
        z = h[q] @ m.W[1].astype(np.float64).T + m.bias[1]
        assert np.allclose(r64["logits"][q], z[r64["logit_ids"][q]], rtol=1e-10, atol=1e-12)
        # prediction = best among the computed outputs only
        assert r64["pred"][q] == r64["logit_ids"][q][np.argmax(r64["logits"][q])]
    # the gathered operand list (ids ascending) reproduces the dense pre-activation
    for q in range(3):
        for n in range(Hd):
            z64 = float(dense[q] @ m.W[0][n].astype(np.float64) + m.bias[0][n])
            z32 = orc.dot_canon32(m.W[0][n][ids[q]], vals[q], 1, m.bias[0][n])
            assert abs(z32 - z64) <= 1e-5 * max(1.0, abs(z64))


def test_canon32_and_ref64_decisions_agree_on_c1_like_workload():
    from paper_2204_08400_b200 import workloads as wl
    w = wl.load("c1", n_queries=256, n_cal=2048, budget_bp=2500)
    m = orc.OracleModel(w.dims, w.has_act, w.W_f32, w.bias, V=w.V, K=w.K, L=w.L)
    m.build(calib_dense=w.calib, seed=w.seed)
    a = m.run(w.budget_bp, x_dense=w.x, mode=orc.CANON32)
    b = m.run(w.budget_bp, x_dense=w.x, mode=orc.REF64)
    agree = np.all(a["codes"] == b["codes"], axis=(1, 2))
    assert agree.mean() > 0.99
    la, lb = a["logits"][agree].astype(np.float64), b["logits"][agree]
    rel = np.max(np.abs(la - lb), axis=1) / np.maximum(np.max(np.abs(lb), axis=1), 1e-30)
    assert rel.max() < 1e-5
    assert np.array_equal(a["pred"][agree], b["pred"][agree])


def test_zero_preactivation_gives_a_zero_hash_bit():
    # FreeHash (Def. 2) is a sign; a pre-activation of exactly 0 is "not active", as for ReLU
    rng = np.random.default_rng(50)
    m = tiny_model(rng, [12, 24, 4], [1, 0], K=3, L=2, bias_scale=0.0)
    m.build(calib_dense=relu_inputs(rng, 80, 12), seed=6)
    x = np.zeros((3, 12), np.float32)                      # every pre-activation is exactly 0
    for mode in (orc.CANON32, orc.REF64):
        r = m.run(np.full(3, 2500, np.uint16), x_dense=x, mode=mode)
        assert np.all(r["codes"] == 0)
    # and a strictly positive one sets it
    hn = m.hash_nodes(0)
    x1 = np.zeros((1, 12), np.float32)
    x1[0] = m.W[0][hn[0, 1]]                               # x parallel to hash function 1 of table 0
    r = m.run(np.full(1, 2500, np.uint16), x_dense=x1)
    assert (int(r["codes"][0, 0, 0]) >> 1) & 1 == 1


def test_prediction_takes_the_lowest_id_among_equal_logits():
    rng = np.random.default_rng(51)
    m = tiny_model(rng, [10, 14, 6], [0, 0], K=2, L=1)
    m.W[1][4] = m.W[1][1]; m.bias[1][4] = m.bias[1][1]      # outputs 1 and 4 are the same function
    m.W[1][5] = m.W[1][1]; m.bias[1][5] = m.bias[1][1]
    x = relu_inputs(rng, 40, 10)
    for mode in (orc.CANON32, orc.REF64):
        r = m.run(np.full(40, 10000, np.uint16), x_dense=x, mode=mode)
        lg = r["logits"]
        assert np.array_equal(lg[:, 1], lg[:, 4])
        top_is_tied = np.argmax(lg, axis=1) == 1
        assert top_is_tied.sum() >= 3                       # the tie decides the prediction for some inputs
        assert np.array_equal(r["pred"], np.argmax(lg, axis=1).astype(np.uint32))   # numpy: first maximum
        assert not np.any(np.isin(r["pred"], [4, 5]))
