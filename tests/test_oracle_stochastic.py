"""Pins for the oracle of the stochastic variant (Appendix B, "Causality under Rejection Sampling"): the shifted
score of Eq. 7, the causal early-stopping frontier scan, and rejection-sampling acceptance.

What fixes them from outside: the appendix's two-token example (0.55 against p(A) = 0.5), the non-anticipation
property the appendix proves (changing the confidence of a position never changes whether that position is kept),
an independent sort-based restatement of the scan, and the textbook fact that rejection sampling reproduces the
target distribution, checked by quadrature over the random numbers."""
import numpy as np
import torch

from oracle import dcut_oracle as orc


def _bf(a):
    return torch.tensor(np.asarray(a), dtype=torch.float32).to(torch.bfloat16)


def _logits_of(p):
    """bf16 logits whose softmax is p up to bf16 rounding of log p."""
    return _bf(np.log(np.asarray(p, np.float64)))


# ------------------------------------------------------------------------------------ Eq. 7

def test_shifted_scores_are_the_scores_moved_one_depth():
    rng = np.random.default_rng(0)
    conf = rng.random((5, 7)).astype(np.float32)
    conf[2, 3] = 0.0
    conf[4, 0] = 1.5      # clamped to 1
    s, sh = orc.scores(conf), orc.scores_shifted(conf)
    assert np.all(sh[:, 0] == 1.0)
    assert np.array_equal(sh[:, 1:], s[:, :-1])          # bit for bit: same left-to-right fp32 products
    assert np.all(sh[2, 4:] == 0.0) and sh[4, 1] == 1.0


def test_shifted_scores_binary_fractions_exact():
    conf = np.array([[0.5, 0.25, 0.5, 1.0]], np.float32)
    assert list(orc.scores_shifted(conf)[0]) == [1.0, 0.5, 0.125, 0.0625]


# ------------------------------------------------------------------------------------ frontier scan

def _scan_by_sorting(conf, cost):
    """Independent restatement: a request's shifted scores never increase with depth, so the frontier order is the
    global order by (score desc, depth asc, request asc); admit while the objective strictly improves."""
    B, g = conf.shape
    sh = orc.scores_shifted(conf)
    order = sorted(((-float(sh[i, k]), k, i) for i in range(B) for k in range(g)))
    one = 1 << 40
    Q, N = 0, 0
    cur = np.float64(B * one) / np.float64(cost[B])
    depths = np.zeros(B, np.int32)
    for negs, k, i in order:
        q = int(np.floor(np.float64(np.float32(-negs)) * 1099511627776.0))
        obj = np.float64(B * one + Q + q) / np.float64(cost[B + N + 1])
        if not obj > cur:
            break
        assert depths[i] == k          # positions of a request arrive in depth order
        cur, Q, N = obj, Q + q, N + 1
        depths[i] += 1
    return depths, N, B * one + Q, float(cur)


def test_scan_matches_sort_based_restatement():
    rng = np.random.default_rng(1)
    for trial in range(40):
        B, g = int(rng.integers(1, 9)), int(rng.integers(1, 9))
        conf = rng.beta(4, 1.5, (B, g)).astype(np.float32)
        if trial % 5 == 0:
            conf = np.round(conf * 4) / 4                  # many equal scores: exercises the tie rule
        slope = [0.02, 0.2, 1.0, 3.0][trial % 4]
        cost = (5.0 + slope * np.arange(B * (g + 1) + 1)).astype(np.float32)
        ref = orc.select_causal(conf, np.zeros((B, g), np.int32), np.zeros(B, np.int32), np.zeros(B, np.int32), cost)
        depths, N, sum_fixed, obj = _scan_by_sorting(conf.astype(np.float32), cost)
        assert np.array_equal(ref.depths, depths) and ref.n_star == N and ref.sum_fixed == sum_fixed
        assert np.float64(ref.objective).tobytes() == np.float64(obj).tobytes()
        assert ref.closure_ok and int(ref.cu_q[-1]) == B + N


def test_scan_hand_example():
    # B = 2, gamma = 3.  shifted scores: r0 = [1, .5, .25], r1 = [1, .75, .375]; cost(T) = 4 + T
    conf = np.array([[0.5, 0.5, 0.5], [0.75, 0.5, 0.5]], np.float32)
    cost = (4.0 + np.arange(9)).astype(np.float32)
    # order: (1,k1,r0) (1,k1,r1) (.75,k2,r1) (.5,k2,r0) (.375,k3,r1) (.25,k3,r0)
    # obj(N): 2/6=.3333  3/7=.4286  4/8=.5  4.75/9=.5278  5.25/10=.525 -> stop at N = 3
    ref = orc.select_causal(conf, np.zeros((2, 3), np.int32), np.zeros(2, np.int32), np.zeros(2, np.int32), cost)
    assert ref.n_star == 3 and list(ref.depths) == [1, 2]
    assert ref.objective == (4.75 * 2 ** 40) / 9.0 and ref.sum_fixed == int(4.75 * 2 ** 40)   # objective in units of 2^-40


def test_scan_stops_at_first_non_improvement_even_if_a_later_size_is_better():
    # the appendix: early stopping may miss a later optimum when the curve is not unimodal
    conf = np.full((1, 4), 0.9, np.float32)
    cost = np.array([1, 1, 3, 3.01, 3.02, 3.03], np.float32)       # a jump at T = 2, flat afterwards
    ref = orc.select_causal(conf, np.zeros((1, 4), np.int32), np.zeros(1, np.int32), np.zeros(1, np.int32), cost)
    assert ref.n_star == 0                                          # (1 + 1)/3 < 1/1: stop at once
    full = orc.select(conf, np.zeros((1, 4), np.int32), np.zeros(1, np.int32), np.zeros(1, np.int32), cost)
    assert full.n_star == 4                                         # the retrospective argmax sees 1 + .9 + .81 + ... over 3.03


def test_retention_of_a_position_does_not_depend_on_its_own_confidence():
    """Non-anticipation: changing c_{i,k} (what the proposal at depth k turned out to be), or any deeper confidence of
    that request, never changes whether depth k of request i is kept.  The inclusive score of Eq. 3 does not have
    this property, which is the appendix's point."""
    rng = np.random.default_rng(2)
    broke_inclusive = 0
    for trial in range(60):
        B, g = int(rng.integers(2, 6)), int(rng.integers(2, 7))
        conf = rng.beta(3, 1.5, (B, g)).astype(np.float32)
        cost = (3.0 + [0.1, 0.5, 1.5][trial % 3] * np.arange(B * (g + 1) + 1)).astype(np.float32)
        z = (np.zeros((B, g), np.int32), np.zeros(B, np.int32), np.zeros(B, np.int32))
        base = orc.select_causal(conf, *z, cost).depths
        base_inc = orc.select(conf, *z, cost).depths
        for _ in range(6):
            i, k = int(rng.integers(0, B)), int(rng.integers(0, g))     # 0-based depth index k <-> depth k + 1
            alt = conf.copy()
            alt[i, k:] = rng.random(g - k).astype(np.float32)
            d = orc.select_causal(alt, *z, cost).depths
            assert (d[i] >= k + 1) == (base[i] >= k + 1)
            d_inc = orc.select(alt, *z, cost).depths
            broke_inclusive += (d_inc[i] >= k + 1) != (base_inc[i] >= k + 1)
    assert broke_inclusive > 0


# ------------------------------------------------------------------------------------ rejection sampling

def _emit_distribution(p, q, retain, n_u=400):
    """Distribution of the emitted token for a one-position block: the proposal z ~ q is verified when retain(z),
    otherwise the position is skipped and the token is drawn from p.  Quadrature over both uniforms."""
    V = len(p)
    tl, dl = _logits_of(p).view(1, V), _logits_of(q).view(1, 1, V)
    us = (np.arange(n_u) + 0.5) / n_u
    out = np.zeros(V)
    for z in range(V):
        draft = np.array([[z]], np.int32)
        hist = np.zeros(V)
        if retain(z):
            cu = np.array([0, 2], np.int32)
            tl2 = torch.cat([tl, tl])                      # the row after the draft has the same target distribution
            for ua in us:
                for usmp in us[:: n_u // 40]:
                    r = orc.accept_rs(tl2, dl, draft, cu, 1, np.array([[ua]], np.float32), np.array([usmp], np.float32))
                    tok = z if r.accept_len[0] == 1 else int(r.bonus[0])
                    hist[tok] += 1
        else:
            cu = np.array([0, 1], np.int32)
            for usmp in us:
                r = orc.accept_rs(tl, dl, draft, cu, 1, np.array([[0.0]], np.float32), np.array([usmp], np.float32))
                hist[int(r.bonus[0])] += 1
        out += q[z] * hist / hist.sum()
    return out


def test_appendix_two_token_example():
    p, q = np.array([0.5, 0.5]), np.array([0.9, 0.1])
    # retention that looks at the proposal itself (keep it only when q(z) > 0.5): biased, P(A) = 0.9 * 5/9 + 0.1 * 0.5
    biased = _emit_distribution(p, q, lambda z: q[z] > 0.5)
    assert abs(biased[0] - 0.55) < 4e-3
    # retention decided before the proposal is seen: the target distribution comes back
    for keep in (True, False):
        fair = _emit_distribution(p, q, lambda z: keep)
        assert abs(fair[0] - 0.5) < 4e-3


def test_rejection_sampling_reproduces_the_target_on_a_small_vocabulary():
    rng = np.random.default_rng(5)
    p, q = rng.dirichlet(np.ones(5)), rng.dirichlet(np.ones(5))
    out = _emit_distribution(p, q, lambda z: True, n_u=200)
    p_bf = torch.softmax(_logits_of(p).double(), 0).numpy()      # what the oracle sees after bf16 rounding of the logits
    assert np.abs(out - p_bf).max() < 1.5e-2


def test_accept_rs_special_cases():
    V = 6
    rng = np.random.default_rng(6)
    tl = _bf(rng.standard_normal((4, V)))
    draft = np.array([[2, 4, 1]], np.int32)
    cu = np.array([0, 4], np.int32)
    ua, us = np.array([[0.999, 0.999, 0.999]], np.float32), np.array([0.3], np.float32)
    # q == p: the ratio is 1 and every draft is accepted whatever u < 1 is; the bonus is the inverse CDF of p at u
    r = orc.accept_rs(tl, tl[:3].view(1, 3, V), draft, cu, 3, ua, us)
    assert r.accept_len[0] == 3 and r.n_accepted_total == 4 and r.prob[0, 1] == 0.0
    p3 = torch.softmax(tl[3].double(), 0).numpy()
    assert r.bonus[0] == int(np.searchsorted(np.cumsum(p3), 0.3 * p3.sum(), side="right"))
    assert list(r.out_tokens[0]) == [2, 4, 1, int(r.bonus[0])]
    # the target gives the second draft (token 4) almost no mass: rejected there, and the residual excludes token 4
    tl2 = tl.clone()
    tl2[1, 4] = -30.0
    r = orc.accept_rs(tl2, tl[:3].view(1, 3, V), draft, cu, 3, np.full((1, 3), 0.5, np.float32), us)
    assert r.accept_len[0] == 1 and r.bonus[0] != 4 and r.prob[0, 0] < 1e-9 and r.prob[0, 1] > 0
    assert list(r.out_tokens[0]) == [2, int(r.bonus[0]), -1, -1]
    # depth 0: only a draw from the target row
    r = orc.accept_rs(tl, tl[:3].view(1, 3, V), draft, np.array([0, 1], np.int32), 3, ua, np.array([0.0], np.float32))
    assert r.accept_len[0] == 0 and r.bonus[0] == 0
