"""Layer-mask solver (Section 2.2, Eq. 5): pins of the oracle's exhaustive enumeration, and the
library's closed-form solver against it.  Host only."""
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_2508_12407_b200 import binding, build

HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load()


def _golden():
    d = {}
    for line in open(os.path.join(HERE, "golden", "eq5_worked_example.txt")):
        line = line.split("#")[0].strip()
        if ":" in line:
            k, v = line.split(":")
            d[k.strip()] = np.array([float(x) for x in v.split()])
    return d


def test_oracle_enumeration_reproduces_hand_worked_example():
    g = _golden()
    alpha = g["alpha"].reshape(3, 2)
    split = oracle.quantile_split(alpha, 2)
    assert split.ravel().tolist() == g["head_is_retrieval"].astype(int).tolist()
    mask, best, second = oracle.layer_mask_enumerate(alpha, split, 1, 0.5)
    assert mask.tolist() == g["layer_is_retrieval"].astype(int).tolist()
    costs = sorted(g["costs"])
    assert abs(best - costs[0]) < 1e-12 and abs(second - costs[1]) < 1e-12


def test_oracle_cost_written_differently():
    # the same objective written with masses per layer in numpy, all subsets via itertools
    rng = np.random.default_rng(5)
    for L, H, p, om in [(4, 3, 2, 0.3), (6, 2, 3, 0.9), (5, 4, 1, 0.0), (7, 3, 4, 1.0)]:
        alpha = rng.random((L, H))
        split = oracle.quantile_split(alpha, p * H)
        a = (alpha * split).sum(1)
        b = (alpha * (1 - split)).sum(1)
        costs = {T: sum(a[i] for i in T) - om * sum(b[i] for i in range(L) if i not in T)
                 for T in itertools.combinations(range(L), p)}
        T_best = min(costs, key=costs.get)
        mask, best, second = oracle.layer_mask_enumerate(alpha, split, p, om)
        assert sorted(np.nonzero(mask == 0)[0].tolist()) == list(T_best)
        assert abs(best - costs[T_best]) < 1e-12
        assert abs(second - sorted(costs.values())[1]) < 1e-12


def test_quantile_split_properties():
    rng = np.random.default_rng(6)
    alpha = rng.random((8, 4))
    for n_s in (0, 1, 7, 16, 32):
        m = oracle.quantile_split(alpha, n_s)
        assert int((m == 0).sum()) == n_s
        if 0 < n_s < alpha.size:
            assert alpha[m == 0].max() <= alpha[m == 1].min()
        want = np.ones(alpha.size, np.uint8)
        want[np.argsort(alpha.ravel(), kind="stable")[:n_s]] = 0
        assert np.array_equal(m.ravel(), want)


def test_already_exclusive_split_costs_nothing():
    # if the quantile split is layer-exclusive already, keeping it is optimal and free
    alpha = np.array([[0.9, 0.8], [0.1, 0.2], [0.7, 0.95], [0.05, 0.3]])
    split = oracle.quantile_split(alpha, 4)
    assert split.tolist() == [[1, 1], [0, 0], [1, 1], [0, 0]]
    for om in (0.0, 0.4, 1.0):
        mask, best, second = oracle.layer_mask_enumerate(alpha, split, 2, om)
        assert mask.tolist() == [1, 0, 1, 0] and best == 0.0 and second > 0.0
        lm, hm, c = binding.layer_mask_solve(alpha, 2, om)
        assert lm.tolist() == [1, 0, 1, 0] and c == 0.0 and np.array_equal(hm, split)


def test_omega_zero_picks_least_retrieval_mass():
    rng = np.random.default_rng(7)
    alpha = rng.random((9, 4))
    p = 3
    split = oracle.quantile_split(alpha, p * 4)
    a = (alpha * split).sum(1)
    mask, best, _ = oracle.layer_mask_enumerate(alpha, split, p, 0.0)
    assert sorted(np.nonzero(mask == 0)[0].tolist()) == sorted(np.argsort(a)[:p].tolist())
    assert abs(best - np.sort(a)[:p].sum()) < 1e-12


def test_head_order_inside_a_layer_does_not_matter():
    rng = np.random.default_rng(8)
    alpha = rng.random((6, 5))
    perm = alpha[:, rng.permutation(5)]
    for om in (0.1, 0.6):
        m1, c1, _ = oracle.layer_mask_enumerate(alpha, oracle.quantile_split(alpha, 15), 3, om)
        m2, c2, _ = oracle.layer_mask_enumerate(perm, oracle.quantile_split(perm, 15), 3, om)
        assert np.array_equal(m1, m2) and abs(c1 - c2) < 1e-12


@pytest.mark.parametrize("L,H", [(2, 1), (3, 4), (8, 8), (12, 4), (16, 8)])
def test_library_solver_equals_exhaustive_enumeration(L, H):
    rng = np.random.default_rng(100 * L + H)
    for trial in range(4):
        alpha = rng.random((L, H)).astype(np.float32)
        for p in sorted({0, 1, L // 2, L - 1, L}):
            for om in (0.0, 0.1, 0.5, 1.0):
                lm, hm, c = binding.layer_mask_solve(alpha, p, om)
                split = oracle.quantile_split(alpha.astype(np.float64), p * H)
                assert np.array_equal(hm, split)
                mask, best, second = oracle.layer_mask_enumerate(alpha.astype(np.float64), split, p, om)
                assert abs(c - best) < 1e-9
                assert int((lm == 0).sum()) == p
                if second - best > 1e-9:          # a unique optimum: the sets must agree
                    assert np.array_equal(lm, mask)


def test_ties_and_errors():
    alpha = np.full((4, 2), 0.5, dtype=np.float32)
    lm, hm, c = binding.layer_mask_solve(alpha, 2, 0.3)
    assert int((lm == 0).sum()) == 2
    _, best, _ = oracle.layer_mask_enumerate(alpha.astype(np.float64), hm, 2, 0.3)
    assert abs(c - best) < 1e-12
    bad = alpha.copy()
    bad[0, 0] = np.nan
    for args in [(bad, 2, 0.3), (alpha, 5, 0.3), (alpha, -1, 0.3), (alpha, 2, 1.5)]:
        with pytest.raises(binding.ZigzagError):
            binding.layer_mask_solve(*args)


def test_paper_scale_solves_instantly():
    # 32 layers, 50 % streaming: the paper's enumeration took minutes; the sort is immediate, and
    # neighbouring omegas often select the same set (Section 3.5 reports that for 0.1 .. 0.4)
    import time
    rng = np.random.default_rng(9)
    alpha = rng.random((32, 8)).astype(np.float32)
    t0 = time.perf_counter()
    masks = [binding.layer_mask_solve(alpha, 16, om)[0] for om in (0.1, 0.2, 0.3, 0.4)]
    assert time.perf_counter() - t0 < 0.5
    for m in masks:
        assert int((m == 0).sum()) == 16
