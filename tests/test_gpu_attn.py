"""dcut_verify_attn against the oracle: |err| <= 1e-2 + 1e-2 |ref| element by element on small
cases spanning several tiles and ragged tails, and on sampled rows at the full workload sizes."""
import numpy as np
import pytest
import torch

from oracle import dcut_oracle as orc
from paper_2607_14647_b200 import workloads as wl
from tests.gpu_helpers import attn_tolerance_ok, dev, make_ctx

pytestmark = pytest.mark.gpu


def _run(cfg, sel, kv, depths, want_lse=True):
    ctx = make_ctx(cfg, max_pages=kv.max_pages_per_req)
    q = wl.q_rows(cfg, depths)
    cu = wl.cu_q_from_depths(depths)
    T = int(cu[-1])
    lse = torch.empty((T, cfg.n_q_heads), dtype=torch.float32, device="cuda") if want_lse else None
    out = ctx.verify_attn(dev(q), dev(kv.k_cache), dev(kv.v_cache), dev(kv.block_table), dev(sel.ctx_lens), dev(cu),
                          cfg.t_cap, lse=lse)
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    ctx.close()
    return q, cu, out.float().cpu().numpy(), None if lse is None else lse.cpu().numpy()


def _full_compare(cfg, sel, kv, depths):
    q, cu, out, lse = _run(cfg, sel, kv, depths)
    ref, ref_lse = orc.verify_attn(q, kv.k_cache, kv.v_cache, kv.block_table, sel.ctx_lens, cu,
                                   cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
    ok, worst = attn_tolerance_ok(out, ref)
    assert ok, f"worst err/limit {worst}"
    np.testing.assert_allclose(lse, ref_lse, rtol=2e-3, atol=2e-3)
    return worst


@pytest.mark.parametrize("depths", [[16, 16, 16, 16], [0, 0, 0, 0], [0, 3, 16, 7], [1, 2, 4, 15]])
def test_tiny_config_every_element(depths):
    cfg = wl.config(0)
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    _full_compare(cfg, sel, kv, np.array(depths, np.int32))


@pytest.mark.parametrize("shape", [dict(n_q_heads=32, n_kv_heads=8, head_dim=128), dict(n_q_heads=16, n_kv_heads=2, head_dim=128),
                                   dict(n_q_heads=8, n_kv_heads=8, head_dim=64), dict(n_q_heads=6, n_kv_heads=2, head_dim=64)])
def test_mid_size_every_element(shape):
    """Contexts from 1 to ~1500 tokens: single-page requests, many chunks, ragged last pages."""
    cfg = wl.custom_config(B=12, gamma=16, ctx_lo=0, ctx_hi=1500, **shape)
    sel = wl.select_inputs(cfg)
    sel.ctx_lens[:4] = [0, 1, 15, 16]                       # degenerate and page-boundary contexts
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    rng = np.random.default_rng(1)
    for depths in (rng.integers(0, 17, cfg.B).astype(np.int32), np.full(cfg.B, 16, np.int32), np.zeros(cfg.B, np.int32)):
        _full_compare(cfg, sel, kv, depths)


@pytest.mark.parametrize("shape,B,gamma,ctx_hi", [
    (dict(n_q_heads=64, n_kv_heads=8, head_dim=128), 5, 16, 1500),     # few requests: cut into chunks, partial results merged
    (dict(n_q_heads=64, n_kv_heads=8, head_dim=128), 40, 16, 400),     # many requests: whole requests per item
    (dict(n_q_heads=16, n_kv_heads=2, head_dim=128), 24, 17, 700),     # 18 tokens x 8 heads = 144 rows: a full 16-row tail
    (dict(n_q_heads=18, n_kv_heads=2, head_dim=128), 10, 15, 900),     # 9 heads per kv head: tails of 7 and 16 rows, ragged groups
])
def test_query_tiles_above_128_rows_every_element(shape, B, gamma, ctx_hi):
    """A request whose (1 + d_i) x (q heads per kv head) query rows exceed the 128 rows of the tensor-memory tile
    (8 heads per kv head at depth 16: 136 rows) stays ONE work item: rows 128.. are computed by the tail warps from
    the same staged pages.  Depths straddle the boundary (127/128/129.. rows), every element against the oracle."""
    cfg = wl.custom_config(B=B, gamma=gamma, ctx_lo=0, ctx_hi=ctx_hi, **shape)
    sel = wl.select_inputs(cfg)
    sel.ctx_lens[:3] = [0, 15, 16]
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    rng = np.random.default_rng(2)
    mixed = rng.integers(max(0, gamma - 3), gamma + 1, cfg.B).astype(np.int32)
    mixed[::5] = rng.integers(0, gamma + 1, len(mixed[::5]))
    for depths in (np.full(cfg.B, gamma, np.int32), mixed):
        _full_compare(cfg, sel, kv, depths)


def test_unused_slots_are_never_read():
    cfg = wl.custom_config(B=6, gamma=16, n_q_heads=8, n_kv_heads=2, head_dim=128, ctx_lo=10, ctx_hi=300)
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    depths = np.array([0, 5, 16, 2, 9, 1], np.int32)
    for i in range(cfg.B):                                  # poison everything past the deepest kept position
        n_slots = ((int(sel.ctx_lens[i]) + cfg.gamma + 1 + 15) // 16) * 16
        for j in range(int(sel.ctx_lens[i]) + int(depths[i]) + 1, n_slots):
            kv.k_cache[kv.block_table[i, j // 16], :, j % 16] = 3.0e4
            kv.v_cache[kv.block_table[i, j // 16], :, j % 16] = 3.0e4
    _full_compare(cfg, sel, kv, depths)


def _sampled_compare(cfg, sel, kv, depths, n_samples, seed=0):
    q, cu, out, lse = _run(cfg, sel, kv, depths)
    T = int(cu[-1])
    rng = np.random.default_rng(seed)
    tok = rng.integers(0, T, n_samples).astype(np.int32)
    head = rng.integers(0, cfg.n_q_heads, n_samples).astype(np.int32)
    # always include the first and last token of the longest and the shortest request
    order = np.argsort(sel.ctx_lens)
    extra = [cu[order[0]], cu[order[0] + 1] - 1, cu[order[-1]], cu[order[-1] + 1] - 1]
    tok[: len(extra)] = extra
    ref, ref_lse = orc.verify_attn(q, kv.k_cache, kv.v_cache, kv.block_table, sel.ctx_lens, cu, cfg.n_q_heads,
                                   cfg.n_kv_heads, cfg.head_dim, cfg.page_size, sample_tok=tok, sample_head=head)
    ok, worst = attn_tolerance_ok(out[tok, head], ref)
    assert ok, f"worst err/limit {worst}"
    np.testing.assert_allclose(lse[tok, head], ref_lse, rtol=2e-3, atol=2e-3)
    assert np.isfinite(out).all()


def _pruned_depths(cfg, sel):
    return orc.select(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens,
                      wl.cost_table_linear(cfg.t_cap + 1, 0.2, 0.0006)).depths


@pytest.mark.parametrize("idx", [1, 2])
def test_full_size_configs_sampled(idx):
    cfg = wl.config(idx)
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    for depths in (_pruned_depths(cfg, sel), np.full(cfg.B, cfg.gamma, np.int32), np.zeros(cfg.B, np.int32)):
        _sampled_compare(cfg, sel, kv, depths, 192)


def test_b256_long_tail_sampled():
    cfg = wl.config(3)
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    _sampled_compare(cfg, sel, kv, _pruned_depths(cfg, sel), 160)
    _sampled_compare(cfg, sel, kv, np.full(cfg.B, cfg.gamma, np.int32), 96, seed=1)
    _sampled_compare(cfg, sel, kv, np.zeros(cfg.B, np.int32), 96, seed=2)


@pytest.mark.parametrize("B,depths", [(8, [3, 16, 0, 8, 12, 1, 5, 16]), (20, [0] * 20), (20, [0, 1, 2, 3, 7] * 4)])
def test_repeated_runs_are_bit_identical(B, depths):
    """The persistent CTAs take work items in whatever order they come free; an item's result must not depend on
    what its CTA worked on before (shallow batches go through the warp-level phase, where it once did)."""
    cfg = wl.custom_config(B=B, gamma=16, n_q_heads=32, n_kv_heads=8, head_dim=128, ctx_lo=100, ctx_hi=3000)
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    depths = np.array(depths, np.int32)
    ctx = make_ctx(cfg, max_pages=kv.max_pages_per_req)
    args = (dev(wl.q_rows(cfg, depths)), dev(kv.k_cache), dev(kv.v_cache), dev(kv.block_table), dev(sel.ctx_lens),
            dev(wl.cu_q_from_depths(depths)), cfg.t_cap)
    first = ctx.verify_attn(*args).clone()
    for _ in range(10):
        assert torch.equal(ctx.verify_attn(*args), first)
    ctx.close()


def test_argument_errors():
    from paper_2607_14647_b200 import binding
    cfg = wl.config(0)
    with pytest.raises(binding.DcutError) as e:
        binding.Context(max_B=4, max_gamma=16, n_q_heads=4, n_kv_heads=1, head_dim=96, max_pages_per_req=4)
    assert e.value.status == binding.EINVAL
    with pytest.raises(binding.DcutError) as e:
        binding.Context(max_B=4, max_gamma=16, n_q_heads=32, n_kv_heads=2, head_dim=128, max_pages_per_req=4)
    assert e.value.status == binding.ECAPACITY                 # 17 * 16 query rows per kv head
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    ctx = make_ctx(cfg, max_pages=kv.max_pages_per_req - 1)
    depths = np.zeros(cfg.B, np.int32)
    with pytest.raises(binding.DcutError) as e:
        ctx.verify_attn(dev(wl.q_rows(cfg, depths)), dev(kv.k_cache), dev(kv.v_cache), dev(kv.block_table),
                        dev(sel.ctx_lens), dev(wl.cu_q_from_depths(depths)), cfg.t_cap)
    assert e.value.status == binding.ECAPACITY
    ctx.close()


@pytest.mark.parametrize("tp", [2, 4])
def test_kv_head_sharding_reproduces_the_unsharded_result(tp):
    """Tensor-parallel sharding of the attention step as the paper's TP deployments would do it: rank r owns kv heads
    r * Hkv/tp .. and their query heads, holds its own slice of the paged cache, and runs the same call on a context
    created for its share of the heads; no exchange inside the step.  Heads are independent, so the concatenated
    shards equal the unsharded output up to rounding: a shard's work is cut into per-SM segments at other places than
    the unsharded call's, so the few items a boundary cuts merge their pieces in a different split (the ranks run one
    after the other here, on one GPU)."""
    cfg = wl.custom_config(B=9, gamma=16, n_q_heads=16, n_kv_heads=4, head_dim=128, ctx_lo=3, ctx_hi=900)
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    depths = np.array([16, 0, 5, 16, 1, 9, 16, 2, 7], np.int32)
    q, cu, full, full_lse = _run(cfg, sel, kv, depths)
    group = cfg.n_q_heads // cfg.n_kv_heads
    hk = cfg.n_kv_heads // tp
    shard_cfg = wl.custom_config(B=cfg.B, gamma=cfg.gamma, n_q_heads=hk * group, n_kv_heads=hk, head_dim=cfg.head_dim,
                                 ctx_lo=cfg.ctx_lo, ctx_hi=cfg.ctx_hi)
    outs = []
    for r in range(tp):
        ctx = make_ctx(shard_cfg, max_pages=kv.max_pages_per_req)
        q_r = q[:, r * hk * group:(r + 1) * hk * group].contiguous()
        k_r = kv.k_cache[:, r * hk:(r + 1) * hk].contiguous()
        v_r = kv.v_cache[:, r * hk:(r + 1) * hk].contiguous()
        out = ctx.verify_attn(dev(q_r), dev(k_r), dev(v_r), dev(kv.block_table), dev(sel.ctx_lens), dev(cu), cfg.t_cap)
        torch.cuda.synchronize()
        assert ctx.poll_device_status() == 0
        ctx.close()
        outs.append(out.float().cpu().numpy())
    got = np.concatenate(outs, axis=1)
    assert np.abs(got - full).max() <= 1e-2 and (got == full).mean() > 0.5       # rounding-level differences, and only in the cut items
    ref, _ = orc.verify_attn(q, kv.k_cache, kv.v_cache, kv.block_table, sel.ctx_lens, cu, cfg.n_q_heads, cfg.n_kv_heads,
                             cfg.head_dim, cfg.page_size)
    ok, worst = attn_tolerance_ok(got, ref)
    assert ok, f"worst err/limit {worst}"


@pytest.mark.parametrize("shallow", [[0, 0], [1, 3], [2]])
def test_a_few_shallow_requests_among_deep_ones(shallow):
    """When the warp-level queue would hold less than an eighth of the pages, the work list sends every item to the
    tcgen05 queue: query tiles of 4 to 16 rows (depth 0 to 3 at four heads per kv head) then run on the 128-row tensor
    memory path.  Every element against the oracle."""
    n = 14
    cfg = wl.custom_config(B=n, gamma=16, n_q_heads=16, n_kv_heads=4, head_dim=128, ctx_lo=200, ctx_hi=1200)
    sel = wl.select_inputs(cfg)
    depths = np.full(n, 16, np.int32)
    order = np.argsort(sel.ctx_lens)                       # the shallow requests get the shortest contexts
    for j, d in enumerate(shallow):
        depths[order[j]] = d
    pages = (sel.ctx_lens + depths + 1 + 15) // 16
    assert 8 * pages[depths < 4].sum() < pages.sum()       # the rule applies
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    _full_compare(cfg, sel, kv, depths)


def test_block_table_entry_outside_the_cache_reads_page_0_and_is_reported():
    """Device status 2.  A block-table entry outside [0, num_pages) must not become an address: the kernel reads
    page 0 in its place, finishes, and the status word says so.  Every other input is valid, so nothing faults; the
    requests whose tables are intact still match the oracle, and the context works normally afterwards."""
    cfg = wl.custom_config(B=6, gamma=16, n_q_heads=8, n_kv_heads=2, head_dim=128, ctx_lo=40, ctx_hi=600)
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    depths = np.array([0, 16, 3, 16, 0, 7], np.int32)         # request 0 runs on the warp-level phase, request 1 on tcgen05
    bad = kv.block_table.copy()
    bad[0, 1] = kv.num_pages + 5                              # past the cache
    bad[1, 0] = -3                                            # negative, in a slot that is in use
    ctx = make_ctx(cfg, max_pages=kv.max_pages_per_req)
    q = wl.q_rows(cfg, depths)
    cu = wl.cu_q_from_depths(depths)
    args = (dev(q), dev(kv.k_cache), dev(kv.v_cache))
    out = ctx.verify_attn(*args, dev(bad), dev(sel.ctx_lens), dev(cu), cfg.t_cap)
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 2
    assert torch.isfinite(out.float()).all()
    # what the kernel computed is the attention over the table with page 0 substituted
    sub = bad.copy()
    sub[0, 1] = 0
    sub[1, 0] = 0
    ref, _ = orc.verify_attn(q, kv.k_cache, kv.v_cache, sub, sel.ctx_lens, cu, cfg.n_q_heads, cfg.n_kv_heads,
                             cfg.head_dim, cfg.page_size)
    ok, worst = attn_tolerance_ok(out.float().cpu().numpy(), ref)
    assert ok, f"worst err/limit {worst}"
    # the status word was cleared by the poll; a valid call on the same context is clean
    out2 = ctx.verify_attn(*args, dev(kv.block_table), dev(sel.ctx_lens), dev(cu), cfg.t_cap)
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    ref2, _ = orc.verify_attn(q, kv.k_cache, kv.v_cache, kv.block_table, sel.ctx_lens, cu, cfg.n_q_heads, cfg.n_kv_heads,
                              cfg.head_dim, cfg.page_size)
    ok, worst = attn_tolerance_ok(out2.float().cpu().numpy(), ref2)
    assert ok, f"worst err/limit {worst}"
    ctx.close()


@pytest.mark.parametrize("B,shape,ctx_lo,ctx_hi,depths_kind", [
    (1, dict(n_q_heads=8, n_kv_heads=1, head_dim=128), 30000, 30000, "full"),     # one item cut into a piece per SM
    (1, dict(n_q_heads=8, n_kv_heads=1, head_dim=128), 30000, 30000, "zero"),
    (2, dict(n_q_heads=32, n_kv_heads=8, head_dim=128), 9000, 20000, "mixed"),    # 16 items, every one cut many times
    (3, dict(n_q_heads=4, n_kv_heads=1, head_dim=64), 4000, 9000, "full"),        # head_dim 64: warp-level pieces with 5 m-tiles
    (480, dict(n_q_heads=8, n_kv_heads=2, head_dim=128), 0, 40, "mixed"),         # many tiny items, several per segment, none cut
])
def test_extreme_batch_shapes_sampled(B, shape, ctx_lo, ctx_hi, depths_kind):
    """The work partition at its extremes: a single long request (one item per kv head, cut into as many pieces as
    there are SMs and merged from that many partial results), and hundreds of one-page requests (segments of many
    whole items).  The selector builds the partition (dcut_enable_plan_in_select)."""
    cfg = wl.custom_config(B=B, gamma=16, ctx_lo=ctx_lo, ctx_hi=ctx_hi, vocab=64, **shape)
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    rng = np.random.default_rng(B)
    depths = {"full": np.full(B, 16, np.int32), "zero": np.zeros(B, np.int32), "mixed": rng.integers(0, 17, B).astype(np.int32)}[depths_kind]
    ctx = make_ctx(cfg, max_pages=kv.max_pages_per_req)
    ctx.enable_plan_in_select(True)
    # force the selector to these depths: confidences 1 on the kept drafts, 0 beyond, and a flat cost
    conf = np.zeros((B, 16), np.float32)
    for i, d in enumerate(depths):
        conf[i, :d] = 1.0
    ctx.set_cost_buckets(B, 16, [int(depths.sum()) + B], [1.0])
    so = ctx.select(dev(conf), dev(sel.draft_ids), dev(sel.bonus_ids), dev(sel.ctx_lens))
    assert np.array_equal(so.depths.cpu().numpy(), depths)
    q = wl.q_rows(cfg, depths)
    cu = wl.cu_q_from_depths(depths)
    T = int(cu[-1])
    lse = torch.empty((T, cfg.n_q_heads), dtype=torch.float32, device="cuda")
    out = ctx.verify_attn(dev(q), dev(kv.k_cache), dev(kv.v_cache), dev(kv.block_table), dev(sel.ctx_lens), so.cu_q, cfg.t_cap, lse=lse)
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    out2 = ctx.verify_attn(dev(q), dev(kv.k_cache), dev(kv.v_cache), dev(kv.block_table), dev(sel.ctx_lens), so.cu_q, cfg.t_cap)
    assert torch.equal(out, out2)                                   # same partition, same bits
    ctx.close()
    n = min(T * cfg.n_q_heads, 96)
    tok = rng.integers(0, T, n).astype(np.int32)
    head = rng.integers(0, cfg.n_q_heads, n).astype(np.int32)
    tok[:2] = [0, T - 1]
    ref, ref_lse = orc.verify_attn(q, kv.k_cache, kv.v_cache, kv.block_table, sel.ctx_lens, cu, cfg.n_q_heads, cfg.n_kv_heads,
                                   cfg.head_dim, cfg.page_size, sample_tok=tok, sample_head=head)
    got = out.float().cpu().numpy()
    ok, worst = attn_tolerance_ok(got[tok, head], ref)
    assert ok, f"worst err/limit {worst}"
    np.testing.assert_allclose(lse.cpu().numpy()[tok, head], ref_lse, rtol=2e-3, atol=2e-3)
    assert np.isfinite(got).all()
