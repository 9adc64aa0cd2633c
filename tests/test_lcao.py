"""LCAO budget choice (Eq. 3): oracle pins on the CPU, device parity on the GPU."""
import numpy as np
import pytest

from oracle import oracle as orc


def test_oracle_lcao_hand_cases():
    bp = np.array([500, 1000, 2500, 5000, 10000], np.uint16)
    ms = np.array([1.0, 2.0, 4.0, 8.0, 16.0], np.float32)
    t0 = np.array([0.0, 0.5, 0.0, 3.0, 0.0, 10.0], np.float32)
    tau = np.array([16.0, 4.5, 3.9, 4.0, 0.5, 10.9], np.float32)
    got, ok = orc.lcao_budgets(bp, ms, t0, tau)
    # 16 fits everything; 0.5+4 <= 4.5; 2 <= 3.9 < 4; 3+1 <= 4; nothing fits 0.5; 10+1 > 10.9
    assert got.tolist() == [10000, 2500, 1000, 500, 500, 500]
    assert ok.tolist() == [1, 1, 1, 1, 0, 0]


def test_oracle_lcao_is_the_brute_force_maximum_and_monotone_in_the_target():
    rng = np.random.default_rng(3)
    bp = rng.permutation(np.arange(100, 10001, 100)).astype(np.uint16)[:40]      # any order
    ms = (bp.astype(np.float32) / 1000.0 + rng.random(40).astype(np.float32))     # not monotone
    t0 = rng.random(500).astype(np.float32) * 3
    tau = rng.random(500).astype(np.float32) * 14
    got, ok = orc.lcao_budgets(bp, ms, t0, tau)
    for q in range(500):
        fits = [int(b) for b, m in zip(bp, ms) if np.float32(t0[q] + m) <= tau[q]]
        assert (ok[q] == 1) == bool(fits)
        assert got[q] == (max(fits) if fits else bp.min())
    looser, _ = orc.lcao_budgets(bp, ms, t0, tau + 1.0)
    assert np.all(looser[ok == 1] >= got[ok == 1])


@pytest.mark.gpu
def test_device_lcao_matches_the_oracle():
    import torch
    from paper_2204_08400_b200 import binding as sl, harness
    rng = np.random.default_rng(4)
    dev = torch.device("cuda:0")
    bp = rng.permutation(np.arange(100, 10001, 100)).astype(np.uint16)[:37]
    ms = (bp.astype(np.float32) / 900.0 + rng.random(37).astype(np.float32))
    n = 10007
    t0 = (rng.random(n) * 3).astype(np.float32)
    tau = (rng.random(n) * 14).astype(np.float32)
    want, ok = orc.lcao_budgets(bp, ms, t0, tau)
    out = torch.zeros(n, dtype=torch.int16, device=dev)
    feas = torch.zeros(n, dtype=torch.uint8, device=dev)
    sl.slonn_lcao_budgets(harness._dev(bp, dev), harness._dev(ms, dev), harness._dev(t0, dev), harness._dev(tau, dev), out, feas)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().view(np.uint16), want)
    assert np.array_equal(feas.cpu().numpy(), ok)
