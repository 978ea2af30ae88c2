"""dcut_accept against the oracle: bit-exact argmax, accepted prefix, bonus and emitted tokens."""
import numpy as np
import pytest
import torch

from oracle import dcut_oracle as orc
from paper_2607_14647_b200 import workloads as wl
from tests.gpu_helpers import dev, make_ctx

pytestmark = pytest.mark.gpu


def _check(ctx, logits, draft_ids, cu_q, gamma, T_cap):
    ref = orc.accept(logits, draft_ids, cu_q, gamma)
    for _ in range(2):      # twice: the per-row scratch must be left clean
        al, bo, toks, total = ctx.accept(dev(logits), dev(draft_ids), dev(cu_q), T_cap)
        torch.cuda.synchronize()
        assert np.array_equal(al.cpu().numpy(), ref.accept_len)
        assert np.array_equal(bo.cpu().numpy(), ref.bonus)
        assert np.array_equal(toks.cpu().numpy(), ref.out_tokens)
        assert int(total.item()) == ref.n_accepted_total
    return ref


def _depth_arms(cfg, sel):
    cost = wl.cost_table_linear(cfg.t_cap + 1, 0.2, 0.0006)
    pruned = orc.select(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens, cost).depths
    return {"pruned": pruned, "full": np.full(cfg.B, cfg.gamma, np.int32), "gamma0": np.zeros(cfg.B, np.int32)}


@pytest.mark.parametrize("idx,arms", [(0, ("pruned", "full", "gamma0")), (1, ("pruned", "full", "gamma0")),
                                      (2, ("pruned", "full", "gamma0")), (3, ("pruned",))])
def test_workload_configs(idx, arms):
    cfg = wl.config(idx)
    sel = wl.select_inputs(cfg)
    ctx = make_ctx(cfg, n_q_heads=0)
    all_arms = _depth_arms(cfg, sel)
    for arm in arms:
        depths = all_arms[arm]
        cu = wl.cu_q_from_depths(depths)
        logits = wl.logits_rows(cfg, sel, depths)
        ref = _check(ctx, logits, sel.draft_ids, cu, cfg.gamma, cfg.t_cap)
        assert np.array_equal(ref.accept_len, np.minimum(sel.reject_index, depths))
        del logits
    ctx.close()


def test_b256_full_depth_on_a_sub_batch():
    """Workload 3 at full depth has 4352 rows of 151 936 logits (1.3 GB): the device scans all of them; the oracle
    checks every fourth request (64 requests, 1088 rows) cut out of the same rows.  Rows are generated per (i, t),
    so a request's rows are the same in the sub-batch."""
    cfg = wl.config(3)
    sel = wl.select_inputs(cfg)
    depths = np.full(cfg.B, cfg.gamma, np.int32)
    cu = wl.cu_q_from_depths(depths)
    logits = wl.logits_rows(cfg, sel, depths)
    ctx = make_ctx(cfg, n_q_heads=0)
    al, bo, toks, total = ctx.accept(dev(logits), dev(sel.draft_ids), dev(cu), cfg.t_cap)
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    al, bo, toks = al.cpu().numpy(), bo.cpu().numpy(), toks.cpu().numpy()
    assert np.array_equal(al, np.minimum(sel.reject_index, depths))            # the planted acceptance, every request
    assert int(total.item()) == int(al.sum()) + cfg.B
    sub = np.arange(0, cfg.B, 4)
    rows = np.concatenate([np.arange(cu[i], cu[i + 1]) for i in sub])
    ref = orc.accept(logits[torch.from_numpy(rows)], sel.draft_ids[sub], wl.cu_q_from_depths(depths[sub]), cfg.gamma)
    assert np.array_equal(al[sub], ref.accept_len) and np.array_equal(bo[sub], ref.bonus)
    assert np.array_equal(toks[sub], ref.out_tokens)
    ctx.close()


def test_ties_nan_inf_signed_zero_rows():
    V = 4099                                   # odd: rows start at every 2-byte alignment
    rng = np.random.default_rng(4)
    T = 64
    x = torch.from_numpy(rng.standard_normal((T, V), dtype=np.float32)).to(torch.bfloat16)
    x[0, 5] = 9.0
    x[0, 4000] = 9.0                           # tie across segments: lowest index
    x[1, :] = float("nan")
    x[2, :] = float("-inf")
    x[3, :] = float("-inf")
    x[3, 77] = float("nan")
    x[3, 78] = -3.0e38
    x[4, :] = -1.0
    x[4, 4098] = -0.0
    x[4, 17] = 0.0
    x[4, 3000] = -0.0
    x[5, :] = float("nan")
    x[5, 4098] = -5.0
    x[6, :] = 2.5                              # every element ties
    x[7, 0] = float("inf")
    x[8, :] = float("nan")
    x[8, 9] = float("-inf")                    # -inf is a value, NaN is not
    for r in range(9, 20):
        x[r, rng.integers(0, V, 8)] = 6.0      # eight-way ties at random places
    cfg = wl.custom_config(B=T, gamma=1, vocab=V)
    ctx = make_ctx(cfg, n_q_heads=0)
    cu = np.arange(T + 1, dtype=np.int32)
    ref = _check(ctx, x, np.zeros((T, 1), np.int32), cu, 1, T)
    assert ref.argmax[:9].tolist() == [5, 0, 0, 78, 17, 4098, 0, 0, 9]
    ctx.close()


@pytest.mark.parametrize("V", [1, 5, 8, 9, 255, 8191, 8193, 32000, 151936])
def test_vocab_sizes_and_alignment(V):
    rng = np.random.default_rng(V)
    B, g = 5, 3
    depths = np.array([3, 0, 2, 1, 3], np.int32)
    cu = wl.cu_q_from_depths(depths)
    T = int(cu[-1])
    x = torch.from_numpy(rng.standard_normal((T, V), dtype=np.float32)).to(torch.bfloat16)
    draft = rng.integers(0, V, size=(B, g)).astype(np.int32)
    for i in range(B):                         # make some drafts match
        for t in range(min(depths[i], 2)):
            x[cu[i] + t, draft[i, t]] = 8.0
    cfg = wl.custom_config(B=B, gamma=g, vocab=V)
    ctx = make_ctx(cfg, n_q_heads=0)
    _check(ctx, x, draft, cu, g, B * (g + 1))
    ctx.close()


def test_unaligned_logits_base():
    V, T = 1001, 7
    rng = np.random.default_rng(9)
    buf = torch.from_numpy(rng.standard_normal(T * V + 3, dtype=np.float32)).to(torch.bfloat16).cuda()
    cfg = wl.custom_config(B=T, gamma=1, vocab=V)
    ctx = make_ctx(cfg, n_q_heads=0)
    for off in (1, 3):
        view = buf[off: off + T * V].view(T, V)
        cu = np.arange(T + 1, dtype=np.int32)
        ref = orc.accept(view.cpu().contiguous(), np.zeros((T, 1), np.int32), cu, 1)
        al, bo, _, _ = ctx.accept(view, dev(np.zeros((T, 1), np.int32)), dev(cu), T)
        assert np.array_equal(bo.cpu().numpy(), ref.bonus)
    ctx.close()


def _past_cap_case():
    """B = 4 requests of 3 rows each (cu_q[B] = 12) handed over with T_cap = 8: the caller's contract is broken.
    Rows 0..7 exist.  Request 2 has rows 6, 7 left (of 6, 7, 8); request 3 has none."""
    V, g = 300, 2
    rng = np.random.default_rng(11)
    x = torch.from_numpy(rng.standard_normal((12, V), dtype=np.float32)).to(torch.bfloat16)
    draft = rng.integers(0, V, size=(4, g)).astype(np.int32)
    for i in range(4):
        for t in range(g):
            x[3 * i + t, draft[i, t]] = 8.0                  # every draft matches wherever its row is looked at
    cu = np.array([0, 3, 6, 9, 12], np.int32)
    am = x.float().argmax(dim=1).numpy()
    want_len = np.array([2, 2, 1, 0], np.int32)             # request 2: row 6 matches, row 7 is its last existing row
    want_bonus = np.array([am[2], am[5], am[7], 0], np.int32)
    return x, draft, cu, g, want_len, want_bonus


def test_cu_q_past_T_cap_is_clamped_and_reported():
    """cu_q[B] > T_cap: rows at or past T_cap are neither read nor cleared, the outputs are defined, and the
    device status word reports code 7.  (Nothing faults: the logits buffer does hold 12 rows.)"""
    x, draft, cu, g, want_len, want_bonus = _past_cap_case()
    cfg = wl.custom_config(B=4, gamma=g, vocab=x.shape[1])
    ctx = make_ctx(cfg, n_q_heads=0)
    al, bo, toks, total = ctx.accept(dev(x), dev(draft), dev(cu), 8)
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 7
    assert np.array_equal(al.cpu().numpy(), want_len) and np.array_equal(bo.cpu().numpy(), want_bonus)
    assert int(total.item()) == int(want_len.sum()) + 4
    # the context is still good and its scratch clean: a valid call right after gives the oracle's answer
    _check(ctx, x, draft, cu, g, 12)
    assert ctx.poll_device_status() == 0
    ctx.close()
