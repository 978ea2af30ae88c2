"""Stochastic variant on the GPU against the oracle: dcut_select_causal bit for bit (shifted scores, early-stopping
scan, packing), dcut_accept_rs on every decision the arithmetic decides.

dcut_accept_rs evaluates softmax in fp32 and the oracle in fp64.  A draft whose u * q(z) lies within 1e-3 (relative)
of p(z), and a sampled token whose cumulative boundary lies within 1e-4 of u * total, could legitimately fall either
way; the tests check those as "valid" (the GPU's answer is one of the two neighbours) and everything else exactly,
and require that at least 95 % of the requests are decided exactly."""
import numpy as np
import pytest
import torch

from oracle import dcut_oracle as orc
from paper_2607_14647_b200 import binding, workloads as wl
from tests.gpu_helpers import dev, make_ctx

pytestmark = pytest.mark.gpu


def _assert_select_equal(out, ref):
    info = binding.read_info(out.info)
    assert info.n_star == ref.n_star and info.t_total == ref.t_total and info.candidate == ref.candidate
    assert info.sum_fixed == ref.sum_fixed
    assert np.float64(info.objective).tobytes() == np.float64(ref.objective).tobytes()
    assert np.array_equal(out.depths.cpu().numpy(), ref.depths) and np.array_equal(out.cu_q.cpu().numpy(), ref.cu_q)
    T = ref.t_total
    for got, want in ((out.tok_req, ref.tok_req), (out.tok_pos, ref.tok_pos), (out.tok_id, ref.tok_id)):
        g = got.cpu().numpy()
        assert np.array_equal(g[:T], want) and np.all(g[T:] == -1)
    assert out.scores.cpu().numpy().tobytes() == ref.scores.tobytes()


def _run_causal(ctx, sel, cost):
    ctx.set_cost_dense(cost)
    out = ctx.select(dev(sel.conf), dev(sel.draft_ids), dev(sel.bonus_ids), dev(sel.ctx_lens), want_scores=True,
                     causal=True)
    torch.cuda.synchronize()
    return out, orc.select_causal(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens, cost)


@pytest.mark.parametrize("index", [0, 1, 2, 3])
def test_select_causal_configs(index):
    cfg = wl.config(index)
    sel = wl.select_inputs(cfg)
    ctx = make_ctx(cfg, vocab=0)
    for slope in (0.0005, 0.002, 0.01, 0.05):
        cost = wl.cost_table_linear(cfg.t_cap + 1, 0.3, slope)
        out, ref = _run_causal(ctx, sel, cost)
        _assert_select_equal(out, ref)
    assert ref.n_star < cfg.B * cfg.gamma       # the steepest table prunes


@pytest.mark.parametrize("B,gamma", [(1, 1), (3, 4), (7, 15), (33, 8), (128, 16), (512, 16)])
def test_select_causal_edge_shapes_and_ties(B, gamma):
    cfg = wl.custom_config(B=B, gamma=gamma, index=200 + B)
    sel = wl.select_inputs(cfg)
    rng = np.random.default_rng(B * 31 + gamma)
    ctx = make_ctx(cfg, vocab=0)
    n = B * (gamma + 1) + 1
    for trial in range(4):
        conf = sel.conf.copy()
        if trial == 1:
            conf = (np.round(conf * 4) / 4).astype(np.float32)          # many equal scores
        if trial == 2:
            conf[rng.random(conf.shape) < 0.1] = 0.0                    # zeroed suffixes
            conf[rng.random(conf.shape) < 0.05] = np.nan
        if trial == 3:
            conf[:] = 1.0                                               # every score 1: order by depth, then request
        sel2 = wl.SelectInputs(conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens, sel.reject_index)
        cost = (1.0 + rng.random() * 0.2 * np.arange(n) + np.where(np.arange(n) > n // 2, 3.0, 0.0)).astype(np.float32)
        out, ref = _run_causal(ctx, sel2, cost)
        _assert_select_equal(out, ref)


def test_select_causal_fixed_budget_is_top_k_of_the_shifted_scores():
    cfg = wl.config(1)
    sel = wl.select_inputs(cfg)
    ctx = make_ctx(cfg, vocab=0)
    K = cfg.B + 77
    ctx.set_cost_buckets(cfg.B, cfg.gamma, [K], [1.0])
    out = ctx.select(dev(sel.conf), dev(sel.draft_ids), dev(sel.bonus_ids), dev(sel.ctx_lens), want_scores=True, causal=True)
    torch.cuda.synchronize()
    sh = orc.scores_shifted(sel.conf)
    order = sorted((-float(sh[i, k]), k, i) for i in range(cfg.B) for k in range(cfg.gamma))
    want = np.zeros(cfg.B, np.int32)
    for _, k, i in order[:77]:
        want[i] += 1
    assert np.array_equal(out.depths.cpu().numpy(), want)
    assert out.scores.cpu().numpy().tobytes() == sh.tobytes()
    ctx.set_cost_buckets(cfg.B, cfg.gamma, [K, K + 10], [1.0, 1.1])       # a retrospective choice among budgets is refused
    with pytest.raises(binding.DcutError):
        ctx.select(dev(sel.conf), dev(sel.draft_ids), dev(sel.bonus_ids), dev(sel.ctx_lens), causal=True)


# ------------------------------------------------------------------------------------ rejection sampling

def _softmax64(bits_row):
    x = bits_row.double().numpy()
    e = np.exp(x - x.max())
    return e / e.sum()


def _check_rs(cfg, V, depths, noise):
    sel = wl.select_inputs(cfg)
    draft = (sel.draft_ids % V).astype(np.int32)
    sel_v = wl.SelectInputs(sel.conf, draft, sel.bonus_ids, sel.ctx_lens, sel.reject_index)
    tl = wl.logits_rows(cfg, sel_v, depths, vocab=V)
    dl = wl.draft_logits_rows(cfg, tl, depths, noise=noise, vocab=V)
    ua, us = wl.uniforms(cfg)
    cu = wl.cu_q_from_depths(depths)
    ctx = make_ctx(cfg, vocab=V)
    al, tok, toks, total, prob = ctx.accept_rs(dev(tl), dev(dl), dev(draft), dev(cu), cfg.t_cap, dev(ua), dev(us),
                                               want_prob=True)
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    al, tok, toks, prob = al.cpu().numpy(), tok.cpu().numpy(), toks.cpu().numpy(), prob.cpu().numpy()
    ref = orc.accept_rs(tl, dl, draft, cu, cfg.gamma, ua, us)
    exact = 0
    for i, d in enumerate(depths):
        # which drafts are decided by the arithmetic (margin), up to the oracle's stopping point
        m_ref = int(ref.accept_len[i])
        decisive = True
        for t in range(min(m_ref + 1, int(d))):
            p, q = _softmax64(tl[cu[i] + t]), _softmax64(dl[i, t])
            z = draft[i, t]
            if abs(float(ua[i, t]) * q[z] - p[z]) <= 1e-3 * p[z]:
                decisive = False
        if decisive:
            assert al[i] == m_ref, (i, al[i], m_ref)
        if al[i] != m_ref:
            continue
        # the sampled token: the oracle's, or a neighbour across a boundary within 1e-4 of u * total
        if m_ref < d:
            p, q = _softmax64(tl[cu[i] + m_ref]), _softmax64(dl[i, m_ref])
            w = np.maximum(p - q, 0.0)
            assert abs(prob[i, 0] - ref.prob[i, 0]) <= 2e-3 * ref.prob[i, 0] + 1e-30
            assert abs(prob[i, 1] - ref.prob[i, 1]) <= 2e-3 * ref.prob[i, 1]
        else:
            w = _softmax64(tl[cu[i] + d])
        cdf = np.cumsum(w)
        target = float(us[i]) * cdf[-1]
        v = int(tok[i])
        assert w[v] > 0.0
        lo = cdf[v - 1] if v > 0 else 0.0
        assert lo - 1e-4 * cdf[-1] <= target <= cdf[v] + 1e-4 * cdf[-1], (i, v, int(ref.bonus[i]))
        assert list(toks[i]) == [int(x) for x in draft[i, :m_ref]] + [v] + [-1] * (cfg.gamma - m_ref)
        exact += v == int(ref.bonus[i])
    assert exact >= int(np.ceil(0.95 * cfg.B))
    assert int(total.item()) == int((al + 1).sum())
    return al, ref


@pytest.mark.parametrize("B,gamma,V", [(4, 4, 37), (9, 8, 1000), (16, 16, 8191), (6, 5, 32000)])
def test_accept_rs_small(B, gamma, V):
    cfg = wl.custom_config(B=B, gamma=gamma, index=300 + B, vocab=V)
    rng = np.random.default_rng(V)
    depths = rng.integers(0, gamma + 1, B).astype(np.int32)
    depths[0], depths[-1] = gamma, 0
    al, ref = _check_rs(cfg, V, depths, noise=0.7)
    assert (al < depths).any() or B < 6      # some rejection happens in these draws


def test_accept_rs_full_vocab_sub_batch():
    cfg = wl.custom_config(B=12, gamma=16, index=2, vocab=151936)
    rng = np.random.default_rng(12)
    depths = rng.integers(0, 17, 12).astype(np.int32)
    _check_rs(cfg, 151936, depths, noise=0.3)


def test_accept_rs_b64_full_vocab():
    """The batch size the benchmark times (B = 64, V = 151 936), ragged depths with both extremes."""
    cfg = wl.custom_config(B=64, gamma=16, index=2, vocab=151936)
    rng = np.random.default_rng(64)
    depths = rng.integers(0, 17, 64).astype(np.int32)
    depths[:4] = [16, 0, 16, 1]
    _check_rs(cfg, 151936, depths, noise=0.3)


def test_accept_rs_identical_distributions_accept_everything():
    cfg = wl.custom_config(B=5, gamma=6, index=305, vocab=500)
    sel = wl.select_inputs(cfg)
    depths = np.array([6, 3, 0, 1, 6], np.int32)
    draft = (sel.draft_ids % 500).astype(np.int32)
    tl = wl.logits_rows(cfg, wl.SelectInputs(sel.conf, draft, sel.bonus_ids, sel.ctx_lens, sel.reject_index), depths, vocab=500)
    cu = wl.cu_q_from_depths(depths)
    dl = torch.zeros((5, 6, 500), dtype=torch.bfloat16)
    for i, d in enumerate(depths):
        for t in range(int(d)):
            dl[i, t] = tl[cu[i] + t]
    ua = np.full((5, 6), 0.999, np.float32)
    us = np.linspace(0.05, 0.95, 5).astype(np.float32)
    ctx = make_ctx(cfg, vocab=500)
    al, tok, toks, total, _ = ctx.accept_rs(dev(tl), dev(dl), dev(draft), dev(cu), cfg.t_cap, dev(ua), dev(us))
    torch.cuda.synchronize()
    assert np.array_equal(al.cpu().numpy(), depths) and int(total.item()) == int(depths.sum()) + 5
    ref = orc.accept_rs(tl, dl, draft, cu, 6, ua, us)
    assert np.array_equal(ref.accept_len, depths)
