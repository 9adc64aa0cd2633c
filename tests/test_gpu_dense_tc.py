"""The tensor-core dense layer (all nodes of a layer computed) against a float64 matrix
product of the same bf16-rounded operands."""
import numpy as np
import pytest

from paper_2204_08400_b200 import workloads as wl_mod

pytestmark = pytest.mark.gpu


def run_dense(M, N, D, relu, seed):
    import torch
    from paper_2204_08400_b200 import binding as sl, harness
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((M, D), dtype=np.float32)
    w = rng.standard_normal((N, D), dtype=np.float32) / np.float32(np.sqrt(D))
    b = rng.standard_normal(N, dtype=np.float32)
    xb, wb = wl_mod.f32_to_bf16_bits(x), wl_mod.f32_to_bf16_bits(w)
    want = wl_mod.bf16_bits_to_f32(xb).astype(np.float64) @ wl_mod.bf16_bits_to_f32(wb).astype(np.float64).T + b
    if relu:
        want = np.maximum(want, 0)
    dev = torch.device("cuda:0")
    dx, dw, db = harness._dev(xb, dev), harness._dev(wb, dev), harness._dev(b, dev)
    out = torch.full((M, N), -7.0, dtype=torch.float32, device=dev)
    outb = torch.zeros((M, N), dtype=torch.int16, device=dev)
    status = torch.ones(4, dtype=torch.int32, device=dev)
    sl.slonn_dense_layer(dx, dw, db, M, N, D, relu, out_f32=out, out_bf16=outb, status=status)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    got = out.cpu().numpy().astype(np.float64)
    scale = np.max(np.abs(want), axis=1, keepdims=True) + 1e-30
    assert np.max(np.abs(got - want) / scale) < 1e-5
    gotb = wl_mod.bf16_bits_to_f32(outb.cpu().numpy().view(np.uint16))
    assert np.array_equal(gotb, wl_mod.bf16_bits_to_f32(wl_mod.f32_to_bf16_bits(out.cpu().numpy())))


@pytest.mark.parametrize("M,N,D,relu", [
    (128, 128, 64, False),       # one tile, one K step
    (128, 128, 256, True),       # full ring of stages
    (256, 384, 1024, True),      # several tiles, ring wraps four times
    (200, 1000, 4096, False),    # ragged rows and columns (zero-filled tile edges)
    (77, 10, 784, True),         # K tail inside a 64-wide step, tiny N
    (1, 4096, 2048, True),       # a single row
    (100, 40, 128, True),        # narrow layer: 48-column tile, output columns dropped by the tiled store
    (300, 72, 192, False),       # 80-column tile: a second, partly filled 64-column output slab
])
def test_dense_layer_matches_float64_matmul(M, N, D, relu):
    run_dense(M, N, D, relu, seed=M + N + D)


# ---- 100 % budget queries routed to the tensor cores inside slonn_run --------------------------

def check_tc_route(wl, kernel_path):
    import sys, os
    sys.path.insert(0, os.path.dirname(__file__))
    from oracle import oracle as orc
    from paper_2204_08400_b200 import binding as sl, harness
    from parity_util import oracle_model, oracle_run
    dm = harness.DeviceModel(wl)
    om = oracle_model(wl)
    g = harness.run_once(dm, wl.x, wl.budget_bp, kernel_path=kernel_path, flags=sl.FLAG_DENSE_TC)
    ref = harness.run_once(dm, wl.x, wl.budget_bp, kernel_path=kernel_path)          # canonical kernels only
    o64 = oracle_run(om, wl, wl.x, wl.budget_bp, orc.REF64)
    assert g["status"][0] == 0
    full = wl.budget_bp == 10000
    assert 0 < full.sum() < full.size
    n_act = sum(wl.has_act)
    ip = g["active_indptr"].astype(np.int64)
    assert np.array_equal(g["active_indptr"], ref["active_indptr"])
    # queries below 100 %: untouched by the flag, bit for bit
    for q in np.nonzero(~full)[0]:
        s, e = ip[q * n_act], ip[q * n_act + n_act]
        assert np.array_equal(g["active_ids"][s:e], ref["active_ids"][s:e])
        assert np.array_equal(g["active_vals"][s:e], ref["active_vals"][s:e])
        assert np.array_equal(g["logits"][q], ref["logits"][q]) and g["pred"][q] == ref["pred"][q]
        assert np.array_equal(g["codes"][q], ref["codes"][q])
    # queries at 100 %: every node active, values and logits within the bf16 tolerance of the fp64 oracle
    worst = 0.0
    code_same = 0
    for q in np.nonzero(full)[0]:
        s, e = ip[q * n_act], ip[q * n_act + n_act]
        assert np.array_equal(g["active_ids"][s:e], ref["active_ids"][s:e])            # all nodes, ascending
        want = o64["logits"][q]
        err = np.max(np.abs(g["logits"][q].astype(np.float64) - want)) / np.max(np.abs(want))
        worst = max(worst, float(err))
        margin = np.sort(want)[-1] - np.sort(want)[-2]
        if margin > 0.05 * np.max(np.abs(want)):
            assert g["pred"][q] == o64["pred"][q]
        v64 = o64["active_vals"][s:e]
        assert np.max(np.abs(g["active_vals"][s:e] - v64)) <= 2e-2 * max(np.max(np.abs(v64)), 1e-30)
        code_same += int(np.array_equal(g["codes"][q], o64["codes"][q]))
    assert worst <= 2e-2, worst
    assert code_same >= 0.9 * full.sum()     # a code bit decided by a near-zero sum may differ
    dm.free()


@pytest.mark.parametrize("kernel_path", [1, 2])
def test_full_budget_queries_on_tensor_cores_narrow(kernel_path):
    wl = wl_mod.load("c5", n_queries=700, n_cal=512, dims=[512, 1024, 1024, 200])
    check_tc_route(wl, kernel_path)


def test_full_budget_queries_on_tensor_cores_wide():
    wl = wl_mod.load("c5", n_queries=300, n_cal=256, dims=[2048, 4096, 4096, 1000])
    check_tc_route(wl, 0)


def test_a_wait_that_runs_out_is_reported_and_leaves_the_device_usable():
    # one-tile problem; the loader's first wait is on a barrier nothing signals and gives up after a few hundred
    # polls, before any copy or product was issued: the launch must end by itself, report SLONN_ERR_TIMEOUT in
    # status[0], leave the output untouched, and the next launch (hook cleared) must compute as usual
    import torch
    from paper_2204_08400_b200 import binding as sl, harness
    dev = torch.device("cuda:0")
    M = N = 128
    D = 64
    rng = np.random.default_rng(7)
    xb = wl_mod.f32_to_bf16_bits(rng.standard_normal((M, D), dtype=np.float32))
    wb = wl_mod.f32_to_bf16_bits(rng.standard_normal((N, D), dtype=np.float32))
    dx, dw = harness._dev(xb, dev), harness._dev(wb, dev)
    out = torch.full((M, N), -7.0, dtype=torch.float32, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    sl.slonn_test_tc_wait_limit(300)
    try:
        sl.slonn_dense_layer(dx, dw, None, M, N, D, False, out_f32=out, status=status)
        torch.cuda.synchronize()
    finally:
        sl.slonn_test_tc_wait_limit(0)
    assert int(status[0]) == -sl.ERR["TIMEOUT"]
    assert bool((out == -7.0).all())
    sl.slonn_dense_layer(dx, dw, None, M, N, D, False, out_f32=out, status=status)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    want = wl_mod.bf16_bits_to_f32(xb).astype(np.float64) @ wl_mod.bf16_bits_to_f32(wb).astype(np.float64).T
    assert np.max(np.abs(out.cpu().numpy() - want)) < 1e-4 * np.max(np.abs(want))
