"""dcut_select against the oracle: bit-exact scores, ranks, cut, depths and packing metadata."""
import numpy as np
import pytest
import torch

from paper_2607_14647_b200 import workloads as wl
from tests.gpu_helpers import assert_select_equal, dev, make_ctx, select_both

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_workload_configs_dense(idx):
    cfg = wl.config(idx)
    sel = wl.select_inputs(cfg)
    ctx = make_ctx(cfg)
    tables = [wl.cost_table_for(cfg), wl.cost_table_linear(cfg.t_cap + 1, 0.2, 0.001),
              wl.cost_table_linear(cfg.t_cap + 1, 0.2, 0.00005), np.full(cfg.t_cap + 1, 1.0, np.float32),
              (1.0 + 10.0 * np.maximum(0, np.arange(cfg.t_cap + 1) - cfg.B)).astype(np.float32)]
    seen = set()
    for cost in tables:
        out, ref = select_both(ctx, sel, cost=cost)
        assert_select_equal(out, ref)
        seen.add(ref.n_star)
    assert 0 in seen and cfg.B * cfg.gamma in seen and len(seen) >= 3     # gamma=0, full gamma, pruned
    ctx.close()


@pytest.mark.parametrize("idx", [0, 2, 3])
def test_workload_configs_bucket(idx):
    from paper_2607_14647_b200 import binding
    cfg = wl.config(idx)
    sel = wl.select_inputs(cfg)
    ctx = make_ctx(cfg)
    K = [binding.budget_from_ratio(cfg.B, cfg.gamma, n, 4) for n in (1, 2, 3, 4)]
    for costs in ([1.0, 1.6, 2.3, 3.1], [1.0, 1.01, 1.02, 1.03], [1.0, 3.0, 6.0, 9.0]):
        out, ref = select_both(ctx, sel, bucket=(K, costs))
        assert_select_equal(out, ref)
    # a single bucket forces N
    for k in (cfg.B, cfg.B + 1, cfg.B + 37, cfg.t_cap):
        out, ref = select_both(ctx, sel, bucket=([k], [1.0]))
        assert_select_equal(out, ref)
        assert ref.t_total == k
    ctx.close()


def test_ties_and_degenerate_confidences():
    cfg = wl.custom_config(B=48, gamma=16)
    ctx = make_ctx(cfg)
    rng = np.random.default_rng(0)
    sel = wl.select_inputs(cfg)
    cases = []
    cases.append(np.ones((cfg.B, cfg.gamma), np.float32))                             # everything ties at 1
    cases.append(np.full((cfg.B, cfg.gamma), 0.8, np.float32))                        # depth-major ties
    cases.append(np.zeros((cfg.B, cfg.gamma), np.float32))                            # everything 0
    c = rng.choice(np.array([0.0, 0.25, 0.5, 1.0], np.float32), size=(cfg.B, cfg.gamma))
    cases.append(c)                                                                   # many exact ties
    c = rng.uniform(-0.5, 1.5, size=(cfg.B, cfg.gamma)).astype(np.float32)
    c[rng.uniform(size=c.shape) < 0.05] = np.nan
    c[0, 0] = -0.0
    cases.append(c)                                                                   # clamp, NaN, -0
    cases.append(np.full((cfg.B, cfg.gamma), 1.0e-4, np.float32))                     # underflow towards 0 / denormals
    for conf in cases:
        sel.conf = conf
        for cost in (wl.cost_table_linear(cfg.t_cap + 1, 1.0, 0.01), np.ones(cfg.t_cap + 1, np.float32)):
            out, ref = select_both(ctx, sel, cost=cost)
            assert_select_equal(out, ref)
        out, ref = select_both(ctx, sel, bucket=([cfg.B + 100], [2.0]))
        assert_select_equal(out, ref)
    ctx.close()


@pytest.mark.parametrize("B,gamma", [(1, 1), (1, 16), (3, 4), (7, 15), (33, 7), (512, 16), (8192, 1), (31, 33)])
def test_edge_shapes(B, gamma):
    cfg = wl.custom_config(B=B, gamma=gamma, conf_a=4.0, conf_b=2.0, conf_decay=0.9)
    sel = wl.select_inputs(cfg)
    ctx = make_ctx(cfg, n_q_heads=0)
    out, ref = select_both(ctx, sel, cost=wl.cost_table_linear(cfg.t_cap + 1, 0.5, 0.002))
    assert_select_equal(out, ref)
    ctx.close()


def test_repeated_runs_are_bit_identical():
    cfg = wl.config(3)
    sel = wl.select_inputs(cfg)
    ctx = make_ctx(cfg)
    ctx.set_cost_dense(wl.cost_table_linear(cfg.t_cap + 1, 0.2, 0.0004))
    args = (dev(sel.conf), dev(sel.draft_ids), dev(sel.bonus_ids), dev(sel.ctx_lens))
    first = ctx.select(*args, want_ranks=True)
    ref = [t.clone() for t in (first.depths, first.cu_q, first.tok_id, first.ranks, first.info)]
    for _ in range(20):
        o = ctx.select(*args, want_ranks=True)
        for a, b in zip((o.depths, o.cu_q, o.tok_id, o.ranks, o.info), ref):
            assert torch.equal(a, b)
    ctx.close()


def test_errors_are_reported_not_launched():
    from paper_2607_14647_b200 import binding
    cfg = wl.custom_config(B=4, gamma=4)
    sel = wl.select_inputs(cfg)
    ctx = make_ctx(cfg, n_q_heads=0)
    args = (dev(sel.conf), dev(sel.draft_ids), dev(sel.bonus_ids), dev(sel.ctx_lens))
    with pytest.raises(binding.DcutError) as e:
        ctx.select(*args)
    assert e.value.status == binding.ECOST                        # no table yet
    ctx.set_cost_dense(np.ones(20, np.float32))
    with pytest.raises(binding.DcutError) as e:
        ctx.select(*args)
    assert e.value.status == binding.ECOST                        # needs 21 entries
    for bad in (0.0, -1.0, np.nan, np.inf):
        t = np.ones(21, np.float32)
        t[7] = bad
        with pytest.raises(binding.DcutError) as e:
            ctx.set_cost_dense(t)
        assert e.value.status == binding.ECOST
    with pytest.raises(binding.DcutError) as e:
        ctx.set_cost_buckets(4, 4, [3, 8], [1.0, 2.0])            # K < B
    assert e.value.status == binding.EINVAL
    with pytest.raises(binding.DcutError) as e:
        ctx.set_cost_buckets(4, 4, [8, 8], [1.0, 2.0])            # not ascending
    assert e.value.status == binding.EINVAL
    ctx.set_cost_buckets(4, 4, [4, 20], [1.0, 2.0])
    big = wl.select_inputs(wl.custom_config(B=5, gamma=4))
    with pytest.raises(binding.DcutError) as e:
        ctx.select(dev(big.conf), dev(big.draft_ids), dev(big.bonus_ids), dev(big.ctx_lens))
    assert e.value.status == binding.ECAPACITY
    with pytest.raises(binding.DcutError) as e:
        binding.Context(max_B=1024, max_gamma=16)
    assert e.value.status == binding.ECAPACITY
    assert ctx.poll_device_status() == 0
    ctx.close()
