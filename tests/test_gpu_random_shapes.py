"""Seeded random small networks against the oracle: layer counts, widths, activator placement, K, L, batch sizes
and budget mixes drawn at random, so that shapes nobody thought of (ragged widths, budgets on both sides of every
kernel-choice threshold, shared-memory sizes near a limit) keep being exercised.  Every case goes through the same
comparison as the named workloads: all kernel families the shape allows, each with the row and the input-stationary
forms forced."""
import numpy as np
import pytest

from paper_2204_08400_b200 import workloads as wl_mod
from test_gpu_parity import check, custom_workload

pytestmark = pytest.mark.gpu

BUDGETS = [50, 300, 500, 1000, 1250, 1300, 1500, 2000, 2100, 2500, 3500, 3600, 3750, 3800, 5000, 7500, 9999, 10000]


def draw_case(seed):
    rng = np.random.default_rng(seed)
    dtype = str(rng.choice(["f32", "bf16"]))
    mult = 4 if dtype == "f32" else 8            # weight rows are whole 16-byte chunks
    n_layers = int(rng.integers(1, 5))
    hi = 2500 if rng.random() < 0.3 else 400
    dims = [(int(rng.integers(8, hi)) // mult + 1) * mult for _ in range(n_layers)] + [int(rng.integers(2, hi))]
    has_act = [int(rng.random() < 0.8) for _ in range(n_layers)]
    if rng.random() < 0.5:
        has_act[-1] = 0
    K = int(rng.integers(1, 11))
    L = int(rng.integers(1, 4))
    while K * L > 32:
        K -= 1
    for l in range(n_layers):                    # an activator layer needs room for its K*L hash nodes
        if has_act[l] and dims[l + 1] < 2 * K * L + 4:
            has_act[l] = 0
    n = int(rng.choice([1, 3, 37, 64, 150, 300, 520, 700]))
    budgets = tuple(sorted(set(int(v) for v in rng.choice(BUDGETS, size=int(rng.integers(1, 6))))))
    return dict(dims=dims, has_act=has_act, dtype=dtype, n=n, n_cal=int(rng.choice([50, 300, 900])), K=K, L=L,
                budgets=budgets, law=str(rng.choice(["relu_normal", "u01_half_zero"])),
                free_hash_nodes=bool(rng.random() < 0.25))


@pytest.mark.parametrize("seed", range(7000, 7048))
def test_random_network_matches_the_oracle(seed):
    c = draw_case(seed)
    wl = custom_workload(seed, c["dims"], c["has_act"], c["dtype"], n=c["n"], n_cal=c["n_cal"], K=c["K"], L=c["L"],
                         budgets=c["budgets"], law=c["law"])
    wl.free_hash_nodes = c["free_hash_nodes"]
    check(wl)


@pytest.mark.parametrize("seed", range(7100, 7112))
def test_random_network_with_csr_first_layer_matches_the_oracle(seed):
    rng = np.random.default_rng(seed)
    dims = [int(rng.integers(300, 20000)), int(rng.integers(8, 64)) * 4, int(rng.integers(200, 70000))]
    n = int(rng.choice([1, 5, 64, 256, 300]))
    wl = wl_mod.load("c3", n_queries=n, n_cal=int(rng.choice([64, 300])), budget_bp=1000, dims=dims,
                     free_hash_nodes=bool(rng.random() < 0.3))
    wl.budget_bp = wl_mod.draw_mixed_budgets(n, seed, (100, 500, 1000, 5000, 10000))
    check(wl)
