"""Pins for the CPU oracle: what the paper and plain mathematics fix, checked
without a GPU.  Each test names the passage or fact it pins."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line


# ---------------------------------------------------------------------------
# small helpers written independently of the oracle
# ---------------------------------------------------------------------------

def rn32(fr: Fraction) -> Fraction:
    """Round an exact rational to the nearest fp32 (ties to even), normal range."""
    if fr == 0:
        return Fraction(0)
    s = -1 if fr < 0 else 1
    a = abs(fr)
    e = 0
    while a >= 2 ** 24:
        a /= 2; e += 1
    while a < 2 ** 23:
        a *= 2; e -= 1
    fl = a.numerator // a.denominator
    rem = a - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return s * Fraction(fl) * (Fraction(2) ** e)


def canon32_exact(w, x, V, bias):
    """The summation contract in exact rational arithmetic with one rounding per step."""
    acc = [Fraction(0)] * 32
    for j in range(len(w)):
        p = (j // V) % 32
        acc[p] = rn32(Fraction(float(w[j])) * Fraction(float(x[j])) + acc[p])
    off = 16
    while off >= 1:
        for p in range(off):
            acc[p] = rn32(acc[p] + acc[p + off])
        off //= 2
    return float(rn32(acc[0] + Fraction(float(bias))))


def tiny_model(rng, dims, has_act, K, L, V=4, bias_scale=0.3, first_sparse=False, list_cap=0):
    W = [rng.standard_normal((dims[l + 1], dims[l])).astype(np.float32) / np.float32(np.sqrt(dims[l]))
         for l in range(len(dims) - 1)]
    b = [(rng.standard_normal(dims[l + 1]) * bias_scale).astype(np.float32) for l in range(len(dims) - 1)]
    return orc.OracleModel(dims, has_act, W, b, V=V, K=K, L=L, list_cap=list_cap, first_sparse=first_sparse)


def dense_forward64(m, x):
    """Plain MLP in float64 with numpy's matrix product."""
    a = x.astype(np.float64)
    for l in range(m.n_layers):
        z = a @ m.W[l].astype(np.float64).T + m.bias[l].astype(np.float64)
        a = z if l == m.n_layers - 1 else np.maximum(z, 0.0)
    return a


# ---------------------------------------------------------------------------
# generator, rounding
# ---------------------------------------------------------------------------

def test_splitmix64_published_vectors():
    for line in _rows("splitmix64.txt"):
        vals = [int(v) for v in line.split()]
        state = vals[0]
        for want in vals[1:]:
            got, state = orc.splitmix64(state)
            assert got == want


def test_budget_rounding_hand_values():
    for line in _rows("budget_nodes.txt"):
        N, bp, B = (int(v) for v in line.split())
        assert orc.budget_nodes(bp, N) == B


# ---------------------------------------------------------------------------
# dot products
# ---------------------------------------------------------------------------

def test_canon32_hand_worked_orderings():
    for line in _rows("canon32_order.txt"):
        head, pairs = line.split("|")
        V, n, bias, want = head.split()
        w = np.zeros(int(n), np.float32)
        for pr in pairs.split():
            i, v = pr.split(":")
            w[int(i)] = np.float32(float(v))
        x = np.ones(int(n), np.float32)
        got = orc.dot_canon32(w, x, int(V), float(bias))
        assert got == float(want), line


def test_canon32_small_integers_are_exact():
    # any summation order gives the exact integer while it stays below 2^24
    rng = np.random.default_rng(5)
    for V in (1, 4, 8):
        for n in (1, 7, 32, 33, 257, 1000):
            w = rng.integers(-9, 10, n).astype(np.float32)
            x = rng.integers(-9, 10, n).astype(np.float32)
            want = int(np.dot(w.astype(np.int64), x.astype(np.int64))) + 3
            assert orc.dot_canon32(w, x, V, 3.0) == float(want)


def test_canon32_matches_exact_rational_emulation():
    rng = np.random.default_rng(6)
    for V in (1, 4, 8):
        for n in (5, 64, 130, 517):
            w = rng.standard_normal(n).astype(np.float32)
            x = rng.standard_normal(n).astype(np.float32)
            b = np.float32(rng.standard_normal())
            assert orc.dot_canon32(w, x, V, b) == canon32_exact(w, x, V, b)


def test_canon32_zero_operands_do_not_change_the_sum():
    # a node that was not computed contributes exactly nothing
    rng = np.random.default_rng(7)
    n = 300
    w = rng.standard_normal(n).astype(np.float32)
    x = rng.standard_normal(n).astype(np.float32)
    x[rng.random(n) < 0.7] = 0.0
    full = orc.dot_canon32(w, x, 4, 0.25)
    # emulate "skip zero entries": same partial assignment, zero terms left out
    acc = [Fraction(0)] * 32
    for j in range(n):
        if x[j] != 0:
            p = (j // 4) % 32
            acc[p] = rn32(Fraction(float(w[j])) * Fraction(float(x[j])) + acc[p])
    off = 16
    while off >= 1:
        for p in range(off):
            acc[p] = rn32(acc[p] + acc[p + off])
        off //= 2
    assert full == float(rn32(acc[0] + Fraction(0.25)))


def test_ref64_dot_is_the_float64_inner_product():
    rng = np.random.default_rng(8)
    w = rng.standard_normal(999).astype(np.float32)
    x = rng.standard_normal(999)
    got = orc.dot_ref64(w, x, 0.5)
    want = float(np.dot(w.astype(np.float64), x) + 0.5)
    assert abs(got - want) <= 1e-12 * max(1.0, abs(want))


# ---------------------------------------------------------------------------
# dense special case: no activator, or a 100 % budget, is the plain MLP
# ---------------------------------------------------------------------------

def test_ref64_without_activators_is_numpy_matmul():
    rng = np.random.default_rng(9)
    m = tiny_model(rng, [24, 40, 16, 5], [0, 0, 0], K=3, L=2)
    x = rng.standard_normal((13, 24)).astype(np.float32)
    r = m.run(np.full(13, 10000, np.uint16), x_dense=x, mode=orc.REF64)
    want = dense_forward64(m, x)
    assert np.max(np.abs(r["logits"] - want)) <= 1e-12 * np.max(np.abs(want))
    assert np.array_equal(r["pred"], np.argmax(want, axis=1).astype(np.uint32))


def test_full_budget_equals_dense_mlp_bit_for_bit():
    # Sec. 3.4: with every node computed nothing differs from the full network
    rng = np.random.default_rng(10)
    dims = [32, 48, 40, 7]
    m = tiny_model(rng, dims, [1, 1, 0], K=3, L=2)
    calib = np.maximum(rng.standard_normal((200, 32)), 0).astype(np.float32)
    m.build(calib_dense=calib, seed=3)
    dense = orc.OracleModel(dims, [0, 0, 0], m.W, m.bias, V=4, K=3, L=2)
    x = np.maximum(rng.standard_normal((17, 32)), 0).astype(np.float32)
    for mode in (orc.CANON32, orc.REF64):
        a = m.run(np.full(17, 10000, np.uint16), x_dense=x, mode=mode)
        b = dense.run(np.full(17, 10000, np.uint16), x_dense=x, mode=mode)
        assert np.array_equal(a["logits"], b["logits"])
        assert np.array_equal(a["pred"], b["pred"])
        ip = a["active_indptr"].astype(np.int64)
        for q in range(17):
            assert np.array_equal(a["active_ids"][ip[2 * q]:ip[2 * q + 1]], np.arange(48))
            assert np.array_equal(a["active_ids"][ip[2 * q + 1]:ip[2 * q + 2]], np.arange(40))


def test_canon32_close_to_ref64_on_dense_network():
    rng = np.random.default_rng(11)
    m = tiny_model(rng, [96, 64, 64, 10], [0, 0, 0], K=3, L=2)
    x = rng.random((50, 96)).astype(np.float32)
    bp = np.full(50, 10000, np.uint16)
    a = m.run(bp, x_dense=x, mode=orc.CANON32)["logits"].astype(np.float64)
    b = m.run(bp, x_dense=x, mode=orc.REF64)["logits"]
    rel = np.max(np.abs(a - b), axis=1) / np.max(np.abs(b), axis=1)
    assert rel.max() < 1e-5
