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
])
def test_dense_layer_matches_float64_matmul(M, N, D, relu):
    run_dense(M, N, D, relu, seed=M + N + D)
