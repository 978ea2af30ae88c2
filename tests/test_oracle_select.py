"""Pins for the selection oracle: what the paper and the arithmetic fix, independent of the
oracle's own code (closed forms, a hand-worked example, brute force, printed table values)."""
import itertools
import json
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import dcut_oracle as orc
from paper_2607_14647_b200 import workloads as wl

TWO40 = float(1 << 40)


def _seq_products_fp32(conf):
    """Prefix products with one fp32 rounding per step, through exact double products
    (a product of two fp32 values is exact in fp64, so the only rounding is the cast)."""
    conf = np.asarray(conf, dtype=np.float32)
    out = np.empty_like(conf)
    for i in range(conf.shape[0]):
        s = np.float32(1.0)
        for k in range(conf.shape[1]):
            s = np.float32(np.float64(s) * np.float64(conf[i, k]))
            out[i, k] = s
    return out


def _dense_select(conf, cost, ctx=None):
    B, g = conf.shape
    z = np.zeros((B, g), np.int32)
    return orc.select(conf, z, np.zeros(B, np.int32), np.zeros(B, np.int32) if ctx is None else ctx, cost)


# ---------------------------------------------------------------- Eq. 3: prefix scores

def test_scores_exact_binary_fractions():
    conf = np.array([[0.5, 0.75, 0.25, 1.0, 0.5], [1.0, 1.0, 0.125, 0.5, 0.75]], np.float32)
    want = np.array([[Fraction(1, 2), Fraction(3, 8), Fraction(3, 32), Fraction(3, 32), Fraction(3, 64)],
                     [1, 1, Fraction(1, 8), Fraction(1, 16), Fraction(3, 64)]], dtype=object)
    got = orc.scores(conf)
    for i in range(2):
        for k in range(5):
            assert Fraction(float(got[i, k])) == want[i, k]


def test_scores_special_cases():
    g = 16
    assert np.all(orc.scores(np.ones((3, g), np.float32)) == 1.0)
    c = np.full((1, g), 0.9, np.float32)
    c[0, 5] = 0.0
    s = orc.scores(c)
    assert np.all(s[0, :5] > 0) and np.all(s[0, 5:] == 0.0)
    # clamp and NaN: >1 counts as 1, <0 and NaN as 0; -0 comes out as +0
    c = np.array([[2.0, 0.5, np.nan, 0.5], [0.5, -3.0, 0.5, 0.5], [-0.0, 0.5, 0.5, 0.5]], np.float32)
    s = orc.scores(c)
    assert s[0].tolist() == [1.0, 0.5, 0.0, 0.0]
    assert s[1].tolist() == [0.5, 0.0, 0.0, 0.0]
    assert not np.signbit(s[2]).any() and np.all(s[2] == 0)


def test_scores_left_to_right_rounding():
    rng = np.random.default_rng(7)
    conf = rng.uniform(0.3, 1.0, size=(64, 16)).astype(np.float32)
    want = _seq_products_fp32(conf)
    got = orc.scores(conf)
    assert got.tobytes() == want.tobytes()
    # the order matters at fp32: a right-to-left product differs somewhere, so this pin
    # would catch a reassociated product
    rl = np.empty_like(conf)
    for k in range(16):
        acc = np.float32(1.0)
        for t in range(k, -1, -1):
            acc = (acc * conf[:, t]).astype(np.float32)
        rl[:, k] = acc
    assert (rl != want).any()


def test_scores_non_increasing():
    sel = wl.select_inputs(wl.config(2))
    s = orc.scores(sel.conf)
    assert np.all(s[:, 1:] <= s[:, :-1])
    assert np.all(s[:, 0] == sel.conf[:, 0])   # p_{i,1} = c_{i,1} exactly


# ---------------------------------------------------------------- Eq. 4: bucket capacity

def test_budget_printed_values(golden_dir):
    g = json.load(open(os.path.join(golden_dir, "cost_table_T3.json")))
    D = g["D"]
    assert [orc.budget(64, D, n, d) for n, d in g["ratios"]] == g["budgets_B64"]
    assert [orc.budget(1, D, n, d) for n, d in g["ratios"]] == g["budgets_B1"]
    # ceil and the lower clamp: B=3, gamma=4 -> total 15: ceil(3.75)=4, ceil(7.5)=8, ceil(11.25)=12, 15
    assert [orc.budget(3, 4, n, d) for n, d in g["ratios"]] == [4, 8, 12, 15]
    assert orc.budget(10, 3, 1, 100) == 10          # max(B, .)
    assert orc.budget(7, 15, 1, 3) == 38            # ceil(112/3) = 38, not 37


# ---------------------------------------------------------------- hand-worked example

def test_hand_example(golden_dir):
    g = json.load(open(os.path.join(golden_dir, "select_hand_example.json")))
    conf = np.array(g["conf"], np.float32)
    B, gam = g["B"], g["gamma"]
    cost = (4 + np.arange(B * (gam + 1) + 1)).astype(np.float32)
    r = _dense_select(conf, cost)
    assert r.scores.tolist() == g["scores"]
    order = sorted(((int(r.ranks[i, k]), i, k + 1) for i in range(B) for k in range(gam)))
    assert [[i, k] for _, i, k in order] == g["ranked_request_depth"]
    assert r.n_star == g["dense"]["n_star"] and r.t_total == B + r.n_star
    assert r.depths.tolist() == g["dense"]["depths"]
    assert r.objective / TWO40 == pytest.approx(g["dense"]["objective"], rel=1e-15)
    assert r.sum_fixed == int((B + g["prefix_sums"][r.n_star]) * (1 << 40))
    assert r.cu_q.tolist() == [0, 1, 3, 5]
    assert r.closure_ok
    rb = orc.select(conf, np.zeros((B, gam), np.int32), np.zeros(B, np.int32), np.zeros(B, np.int32),
                    np.array(g["bucket"]["cost_ms"], np.float32), bucket_K=g["bucket"]["K"])
    assert rb.n_star == g["bucket"]["n_star"] and rb.candidate == g["bucket"]["candidate"]
    assert rb.depths.tolist() == g["bucket"]["depths"]
    assert rb.objective / TWO40 == pytest.approx(g["bucket"]["objective"], rel=1e-15)


# ---------------------------------------------------------------- brute force over depth vectors

@pytest.mark.parametrize("seed", range(12))
def test_brute_force_b3_gamma4(seed):
    """For fixed N the best depth vector is the top-N set (scores are non-increasing in depth),
    so the maximum of (B + sum of kept scores) / cost(B + sum d) over ALL (gamma+1)^B depth
    vectors equals the selector's objective."""
    rng = np.random.default_rng(seed)
    B, g = 3, 4
    conf = rng.beta(3, 1.5, size=(B, g)).astype(np.float32)
    kind = seed % 3
    T = np.arange(B * (g + 1) + 1, dtype=np.float64)
    cost = {0: 4.0 + T, 1: 10.0 + 0.3 * np.maximum(0, T - 5) ** 1.5, 2: 1.0 + 0.05 * T}[kind].astype(np.float32)
    p = _seq_products_fp32(conf)
    best = None
    for d in itertools.product(range(g + 1), repeat=B):
        num = Fraction(B) + sum(Fraction(float(p[i, k])) for i in range(B) for k in range(d[i]))
        obj = num / Fraction(float(cost[B + sum(d)]))
        key = (obj, -sum(d))
        if best is None or key > best[0]:
            best = (key, d)
    r = _dense_select(conf, cost)
    assert r.closure_ok
    assert r.n_star == sum(best[1])
    assert r.depths.tolist() == list(best[1])          # random scores: no ties straddle the cut
    assert r.objective / TWO40 == pytest.approx(float(best[0][0]), rel=1e-9)


# ---------------------------------------------------------------- limiting cost tables

def test_flat_cost_keeps_everything():
    cfg = wl.config(1)
    sel = wl.select_inputs(cfg)
    r = _dense_select(sel.conf, np.full(cfg.t_cap + 1, 3.0, np.float32))
    assert r.n_star == cfg.B * cfg.gamma and np.all(r.depths == cfg.gamma)   # unpruned verification
    assert r.cu_q.tolist() == list(range(0, cfg.t_cap + 1, cfg.gamma + 1))


def test_steep_cost_keeps_only_bonus():
    cfg = wl.config(1)
    sel = wl.select_inputs(cfg)
    cost = (1.0 + 10.0 * np.maximum(0, np.arange(cfg.t_cap + 1) - cfg.B)).astype(np.float32)
    r = _dense_select(sel.conf, cost)
    assert r.n_star == 0 and np.all(r.depths == 0) and r.t_total == cfg.B    # K >= B: one token each
    assert r.sum_fixed == cfg.B << 40


def test_cost_errors():
    conf = np.full((2, 4), 0.5, np.float32)
    with pytest.raises(orc.OracleError):
        _dense_select(conf, np.ones(10, np.float32))                # needs 11 entries
    bad = np.ones(11, np.float32)
    bad[4] = 0.0
    with pytest.raises(orc.OracleError):
        _dense_select(conf, bad)
    bad[4] = np.nan
    with pytest.raises(orc.OracleError):
        _dense_select(conf, bad)


# ---------------------------------------------------------------- uniform confidence closed form + Table 3

@pytest.mark.parametrize("hw,c0,want_bucket", [("H20", 0.8, 0), ("H800", 0.8, 1), ("H20", 0.95, 2),
                                               ("H800", 0.95, 2), ("H20", 0.5, 0), ("H800", 0.5, 0)])
def test_uniform_confidence_with_printed_cost_table(golden_dir, hw, c0, want_bucket):
    """With c_{i,t} = c0 for all i, t the ranking is depth-major, the top-K set is n = K/B full
    levels (bonus included) and Eq. 5 has the closed form B (1 - c0^n) / (1 - c0) / C(B, rho)."""
    g = json.load(open(os.path.join(golden_dir, "cost_table_T3.json")))
    B, D = 64, g["D"]
    cost = np.array(g[hw][g["B"].index(B)], np.float32)
    K = g["budgets_B64"]
    conf = np.full((B, D), c0, np.float32)
    r = orc.select(conf, np.zeros((B, D), np.int32), np.zeros(B, np.int32), np.zeros(B, np.int32), cost, bucket_K=K)
    closed = [B * (1 - c0 ** (k // B)) / (1 - c0) / float(c) for k, c in zip(K, cost)]
    assert int(np.argmax(closed)) == want_bucket
    assert r.candidate == want_bucket
    assert r.objective / TWO40 == pytest.approx(closed[want_bucket], rel=2e-6)
    assert np.all(r.depths == K[want_bucket] // B - 1)


def test_steeper_cost_prunes_more(golden_dir):
    """Section 3.3: heavy pruning when verification is expensive (H20), light when cheap (H800)."""
    g = json.load(open(os.path.join(golden_dir, "cost_table_T3.json")))
    cfg = wl.custom_config(B=64, gamma=15, conf_kind="beta_decay", conf_a=6.0, conf_b=2.0, conf_decay=0.95)
    sel = wl.select_inputs(cfg)
    pick = {}
    for hw in ("H20", "H800"):
        cost = np.array(g[hw][4], np.float32)
        pick[hw] = orc.select(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens, cost,
                              bucket_K=g["budgets_B64"]).t_total
    assert pick["H20"] <= pick["H800"]


# ---------------------------------------------------------------- invariants on the workloads

@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_closure_and_counts_on_workloads(idx):
    cfg = wl.config(idx)
    sel = wl.select_inputs(cfg)
    cost = wl.cost_table_for(cfg)
    r = orc.select(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens, cost)
    assert r.closure_ok
    assert int(r.depths.sum()) == r.n_star and r.t_total == cfg.B + r.n_star == int(r.cu_q[-1])
    # ranks are a permutation and each request's ranks increase with depth (contiguous prefixes)
    assert sorted(r.ranks.ravel().tolist()) == list(range(cfg.B * cfg.gamma))
    assert np.all(np.diff(r.ranks, axis=1) > 0)
    # depth = number of positions ranked below N* = deepest selected position
    sel_mask = r.ranks < r.n_star
    assert np.array_equal(sel_mask.sum(1), r.depths)
    for i in range(cfg.B):
        assert sel_mask[i, : r.depths[i]].all() and not sel_mask[i, r.depths[i]:].any()
    # exact fixed-point sum equals the sum over the selected set; double sum agrees to 1e-8
    fixed = (cfg.B << 40) + int(sum(int(np.floor(float(s) * TWO40)) for s in r.scores[sel_mask]))
    assert fixed == r.sum_fixed
    assert r.sum_fixed / TWO40 == pytest.approx(r.sum_f64, rel=1e-8)
    assert r.objective == pytest.approx(r.sum_fixed / float(cost[r.t_total]), rel=1e-15)
    # packing metadata: request-major, bonus first, positions L_i + t
    for i in range(cfg.B):
        a, b = r.cu_q[i], r.cu_q[i + 1]
        assert np.all(r.tok_req[a:b] == i)
        assert r.tok_pos[a:b].tolist() == list(range(sel.ctx_lens[i], sel.ctx_lens[i] + r.depths[i] + 1))
        assert r.tok_id[a] == sel.bonus_ids[i]
        assert r.tok_id[a + 1:b].tolist() == sel.draft_ids[i, : r.depths[i]].tolist()


def test_objective_is_argmax_over_all_candidates():
    cfg = wl.config(2)
    sel = wl.select_inputs(cfg)
    cost = wl.cost_table_linear(cfg.t_cap + 1, 0.2, 0.001)
    r = orc.select(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens, cost)
    flat = np.sort(r.scores.ravel().astype(np.float64))[::-1]
    S = np.concatenate([[0.0], np.cumsum(flat)])
    obj = (cfg.B + S) / cost[cfg.B: cfg.B + len(S)].astype(np.float64)
    assert abs(int(np.argmax(obj)) - r.n_star) <= 1
    assert obj.max() == pytest.approx(r.objective / TWO40, rel=1e-8)
    assert 0 < r.n_star < cfg.B * cfg.gamma            # this table really prunes


def test_request_permutation_permutes_depths():
    cfg = wl.config(1)
    sel = wl.select_inputs(cfg)
    cost = wl.cost_table_linear(cfg.t_cap + 1, 0.2, 0.002)
    r = orc.select(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens, cost)
    perm = np.random.default_rng(3).permutation(cfg.B)
    r2 = orc.select(sel.conf[perm], sel.draft_ids[perm], sel.bonus_ids[perm], sel.ctx_lens[perm], cost)
    assert r2.n_star == r.n_star and np.array_equal(r2.depths, r.depths[perm])


# ---------------------------------------------------------------- tie rules

def test_ties_depth_then_request():
    B, g = 3, 4
    conf = np.ones((B, g), np.float32)                 # every score equals 1
    K = [B + 5]
    r = orc.select(conf, np.zeros((B, g), np.int32), np.zeros(B, np.int32), np.zeros(B, np.int32),
                   np.ones(1, np.float32), bucket_K=K)
    # depth 1 of requests 0,1,2 first, then depth 2 of requests 0,1
    assert r.depths.tolist() == [2, 2, 1]
    assert r.ranks.tolist() == [[0, 3, 6, 9], [1, 4, 7, 10], [2, 5, 8, 11]]


def test_objective_ties_pick_smallest_n():
    # zero scores beyond the first level: adding them never raises the numerator; with a flat
    # cost the objective is equal for all N >= B, and the cheapest (smallest N) must win
    B, g = 2, 3
    conf = np.array([[0.5, 0.0, 0.5], [0.25, 0.0, 0.5]], np.float32)
    r = _dense_select(conf, np.ones(B * (g + 1) + 1, np.float32))
    assert r.n_star == 2 and r.depths.tolist() == [1, 1]


def test_bucket_equals_dense_when_all_budgets_offered():
    cfg = wl.config(0)
    sel = wl.select_inputs(cfg)
    cost = wl.cost_table_for(cfg)
    rd = orc.select(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens, cost)
    K = list(range(cfg.B, cfg.t_cap + 1))
    rb = orc.select(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens, cost[cfg.B:], bucket_K=K)
    assert rb.n_star == rd.n_star and np.array_equal(rb.depths, rd.depths) and rb.objective == rd.objective


def test_bucket_validation():
    conf = np.full((2, 4), 0.5, np.float32)
    z = np.zeros((2, 4), np.int32)
    zz = np.zeros(2, np.int32)
    for K in ([1, 5], [5, 5], [6, 5], [5, 11]):
        with pytest.raises(orc.OracleError):
            orc.select(conf, z, zz, zz, np.ones(2, np.float32), bucket_K=K)


def test_expected_vs_realised_is_sane():
    """Eq. 2's estimate against the planted acceptance.  Sanity only: parity unpinned."""
    cfg = wl.config(2)
    sel = wl.select_inputs(cfg)
    r = orc.select(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens,
                   wl.cost_table_linear(cfg.t_cap + 1, 0.2, 0.0003))
    realised = int((1 + np.minimum(sel.reject_index, r.depths)).sum())
    assert cfg.B <= realised <= r.t_total
    assert 0.3 < realised / r.sum_f64 < 3.0
