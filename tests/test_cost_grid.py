"""Start-up cost table C(B, rho) (Appendix C; Eq. 4; Table 3): the oracle's plain definitions pinned against the
paper's table and brute force, the library's host calls against the oracle, and the profiler's monotone fit against
its definition.  Host logic only: no GPU."""
import itertools
import json
import os

import numpy as np
import pytest

from oracle import dcut_oracle as orc

T3_B = [1, 8, 16, 32, 64]
RATIOS = [(1, 4), (1, 2), (3, 4), (1, 1)]


@pytest.fixture(scope="module")
def t3(golden_dir):
    return json.load(open(os.path.join(golden_dir, "cost_table_T3.json")))


# ---------------------------------------------------------------------------------------------- oracle pins

def test_oracle_nearest_is_the_brute_force_argmin_with_ties_to_the_larger_batch():
    for sizes in ([1, 8, 16, 32, 64], [4], [2, 3, 10, 11, 40]):
        for B in range(1, 90):
            b = orc.cost_grid_nearest(sizes, B)
            dist = [abs(s - B) for s in sizes]
            assert dist[b] == min(dist)
            assert b == max(i for i, d in enumerate(dist) if d == min(dist))      # tie -> larger captured size
    assert orc.cost_grid_nearest(T3_B, 64) == 4 and orc.cost_grid_nearest(T3_B, 1) == 0
    assert orc.cost_grid_nearest(T3_B, 40) == 3          # |40 - 32| = 8 < |40 - 64| = 24
    assert orc.cost_grid_nearest(T3_B, 48) == 4          # tie between 32 and 64
    assert orc.cost_grid_nearest(T3_B, 12) == 2          # tie between 8 and 16
    assert orc.cost_grid_nearest(T3_B, 1000) == 4


def test_oracle_median_against_numpy_and_by_hand():
    assert orc.cost_grid_median([3.0]) == np.float32(3.0)
    assert orc.cost_grid_median([5.0, 1.0, 3.0]) == np.float32(3.0)
    assert orc.cost_grid_median([4.0, 1.0, 3.0, 2.0]) == np.float32(2.5)
    rng = np.random.default_rng(0)
    for n in range(1, 12):
        x = rng.uniform(0.1, 9, n).astype(np.float32)
        assert abs(float(orc.cost_grid_median(x)) - float(np.median(x.astype(np.float64)))) <= 1e-6


def test_oracle_buckets_reproduce_table_3_rows_and_eq4_budgets(t3):
    for hw in ("H20", "H800"):
        K, c = orc.cost_grid_buckets(t3["B"], t3["ratios"], t3["D"], t3[hw], 64)
        assert K.tolist() == t3["budgets_B64"] and np.allclose(c, t3[hw][4])
        K, c = orc.cost_grid_buckets(t3["B"], t3["ratios"], t3["D"], t3[hw], 1)
        assert K.tolist() == t3["budgets_B1"] and np.allclose(c, t3[hw][0])
        K, c = orc.cost_grid_buckets(t3["B"], t3["ratios"], t3["D"], t3[hw], 40)     # between captured points
        assert K.tolist() == [160, 320, 480, 640] and np.allclose(c, t3[hw][3])      # live budgets, row of B = 32


def test_oracle_buckets_merge_equal_budgets_and_keep_the_cheaper():
    # B = 3, gamma = 1: B(gamma+1) = 6; ratios 1/4 and 1/2 both clamp to K = 3
    K, c = orc.cost_grid_buckets([3], RATIOS, 1, [[5.0, 4.0, 6.0, 7.0]], 3)
    assert K.tolist() == [3, 5, 6] and c.tolist() == [4.0, 6.0, 7.0]


def test_selecting_on_a_table_3_row_picks_the_bucket_the_closed_form_gives(t3):
    """Uniform confidence c0: the top-K is depth-major, so the objective of bucket K = n B is B (1 - c0^n) / (1 - c0) / C;
    with Table 3's B = 64 rows c0 = 0.8 prefers 25 % on H20 and 50 % on H800 (Eq. 5 evaluated by hand)."""
    B, D = 64, t3["D"]
    for hw, c0, want in (("H20", 0.8, 0), ("H800", 0.8, 1), ("H20", 0.95, 2), ("H800", 0.95, 2), ("H20", 0.5, 0), ("H800", 0.5, 0)):
        K, cost = orc.cost_grid_buckets(t3["B"], t3["ratios"], D, t3[hw], B)
        conf = np.full((B, D), c0, np.float32)
        z = np.zeros((B, D), np.int32)
        r = orc.select(conf, z, np.zeros(B, np.int32), np.zeros(B, np.int32), cost, bucket_K=K)
        assert r.candidate == want, (hw, c0, r.candidate)


# ---------------------------------------------------------------------------------------------- library vs oracle

def test_library_grid_matches_the_oracle(t3):
    from paper_2607_14647_b200 import binding
    rng = np.random.default_rng(3)
    for sizes, ratios, gamma in ((t3["B"], [tuple(r) for r in t3["ratios"]], t3["D"]), ([2, 3, 10, 11, 40], [(1, 8), (1, 3), (1, 1)], 4),
                                 ([5], [(1, 1)], 1)):
        g = binding.CostGrid(sizes, ratios, gamma)
        table = np.zeros((len(sizes), len(ratios)), np.float32)
        for b in range(len(sizes)):
            for r in range(len(ratios)):
                samples = rng.uniform(0.2, 30.0, int(rng.integers(1, 9))).astype(np.float32)
                g.record(b, r, samples)
                table[b, r] = orc.cost_grid_median(samples)
        assert np.array_equal(g.table(), table)
        for B in list(range(1, 70)) + [500]:
            assert g.nearest(B) == orc.cost_grid_nearest(sizes, B)
            for r, (num, den) in enumerate(ratios):
                assert g.budget(B, r) == orc.budget(B, gamma, num, den)
            K, c = g.buckets(B)
            Ko, co = orc.cost_grid_buckets(sizes, ratios, gamma, table, B)
            assert np.array_equal(K, Ko) and np.array_equal(c, co)
        g.close()


def test_library_grid_argument_errors():
    from paper_2607_14647_b200 import binding
    for bad in (([8, 8], RATIOS, 4), ([8, 4], RATIOS, 4), ([0], RATIOS, 4), ([4], [(1, 2), (1, 4)], 4), ([4], [(3, 2)], 4),
                ([4], [(1, 2), (2, 4)], 4), ([4], RATIOS, 0)):
        with pytest.raises(binding.DcutError):
            binding.CostGrid(*bad)
    g = binding.CostGrid([4, 8], RATIOS, 4)
    with pytest.raises(binding.DcutError) as e:
        g.buckets(4)                                     # nothing recorded yet
    assert e.value.status == binding.ECOST
    for samples in ([1.0, -2.0], [0.0], [float("nan")], [float("inf")]):
        with pytest.raises(binding.DcutError) as e:
            g.record(0, 0, samples)
        assert e.value.status == binding.ECOST
    with pytest.raises(binding.DcutError):
        g.record(2, 0, [1.0])


# ---------------------------------------------------------------------------------------------- profiler's monotone fit

def _brute_isotonic(y):
    """Isotonic regression by its definition on a tiny input: the best non-decreasing step function whose levels are
    block means, over all ways to cut the sequence into consecutive blocks."""
    n = len(y)
    best = None
    for cuts in itertools.product([0, 1], repeat=n - 1):
        blocks, start = [], 0
        for i, c in enumerate(cuts):
            if c:
                blocks.append((start, i + 1))
                start = i + 1
        blocks.append((start, n))
        fit = np.concatenate([np.full(b - a, np.mean(y[a:b])) for a, b in blocks])
        if np.all(np.diff(fit) >= -1e-12):
            err = float(((fit - y) ** 2).sum())
            if best is None or err < best[0] - 1e-12:
                best = (err, fit)
    return best[1]


def test_isotonic_fit_is_the_least_squares_monotone_fit():
    from paper_2607_14647_b200 import profiler
    rng = np.random.default_rng(1)
    assert np.allclose(profiler.isotonic_non_decreasing([1, 2, 3, 5]), [1, 2, 3, 5])            # already ascending: untouched
    assert np.allclose(profiler.isotonic_non_decreasing([3, 1]), [2, 2])
    assert np.allclose(profiler.isotonic_non_decreasing([1, 3, 2, 4]), [1, 2.5, 2.5, 4])
    assert np.allclose(profiler.isotonic_non_decreasing([5, 4, 3, 2, 1]), [3] * 5)
    for _ in range(30):
        y = rng.uniform(0, 1, int(rng.integers(2, 9))) + np.linspace(0, 1, 1)[0]
        fit = profiler.isotonic_non_decreasing(y)
        assert np.all(np.diff(fit) >= -1e-12)
        assert np.allclose(fit, _brute_isotonic(y))
        assert abs(fit.sum() - y.sum()) < 1e-9                                                    # pooled means keep the total


def test_dense_table_interpolates_the_fitted_points():
    from paper_2607_14647_b200 import profiler
    tab = profiler.dense_table([64, 320, 192, 448], [0.30, 0.29, 0.31, 0.35], 512)                 # unsorted, one violation
    assert tab.dtype == np.float32 and len(tab) == 512 and np.all(np.diff(tab) >= 0) and np.all(tab > 0)
    assert np.isclose(tab[64], 0.30) and np.isclose(tab[192], 0.30) and np.isclose(tab[320], 0.30) and np.isclose(tab[448], 0.35)
    assert np.isclose(tab[0], 0.30) and np.isclose(tab[511], 0.35) and np.isclose(tab[384], 0.325)
