"""The verify step as the benchmark runs it: select -> verify attention -> accept captured ONCE in a CUDA graph and
replayed for different inputs (the packed length is read on the device, so one graph serves every depth vector),
with the attention work list built in the selector's tail (dcut_enable_plan_in_select).  Depths, packing and
acceptance against the oracle bit for bit, attention within 1e-2 + 1e-2 |ref|."""
import numpy as np
import pytest
import torch

from oracle import dcut_oracle as orc
from paper_2607_14647_b200 import workloads as wl
from tests.gpu_helpers import attn_tolerance_ok, dev, make_ctx

pytestmark = pytest.mark.gpu


def _pack_rows(cfg, depths, all_rows):
    idx = np.concatenate([i * (cfg.gamma + 1) + np.arange(d + 1) for i, d in enumerate(depths)])
    return all_rows[torch.from_numpy(idx)]


def _step_state(cfg, kv):
    i32 = dict(dtype=torch.int32, device="cuda")
    cap = cfg.t_cap
    return dict(conf=torch.zeros((cfg.B, cfg.gamma), dtype=torch.float32, device="cuda"),
                q=torch.zeros((cap, cfg.n_q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda"),
                logits=torch.zeros((cap, cfg.vocab), dtype=torch.bfloat16, device="cuda"),
                attn=torch.zeros((cap, cfg.n_q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda"),
                accept_len=torch.zeros(cfg.B, **i32), bonus=torch.zeros(cfg.B, **i32),
                toks=torch.zeros((cfg.B, cfg.gamma + 1), **i32), total=torch.zeros(1, **i32),
                k=dev(kv.k_cache), v=dev(kv.v_cache), bt=dev(kv.block_table))


@pytest.mark.parametrize("shape,B,ctx_hi", [(dict(n_q_heads=32, n_kv_heads=8, head_dim=128), 24, 700),
                                            (dict(n_q_heads=64, n_kv_heads=8, head_dim=128), 10, 900),
                                            (dict(n_q_heads=4, n_kv_heads=1, head_dim=64), 6, 300)])
def test_graph_replayed_step_matches_the_oracle_for_changing_inputs(shape, B, ctx_hi):
    cfg = wl.custom_config(B=B, gamma=16, ctx_lo=5, ctx_hi=ctx_hi, vocab=2048, **shape)
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    full = np.full(cfg.B, cfg.gamma, np.int32)
    q_all = wl.q_rows(cfg, full)
    logits_all = wl.logits_rows(cfg, sel, full)
    cost = wl.cost_table_linear(cfg.t_cap + 1, 0.2, 0.004)
    ctx = make_ctx(cfg, max_pages=kv.max_pages_per_req)
    ctx.set_cost_dense(cost)
    ctx.enable_plan_in_select(True)
    st = _step_state(cfg, kv)
    d_draft, d_bonus, d_ctx = dev(sel.draft_ids), dev(sel.bonus_ids), dev(sel.ctx_lens)
    so = ctx.select(st["conf"].fill_(0.5), d_draft, d_bonus, d_ctx)              # allocates the selector's outputs once

    def step():
        ctx.select(st["conf"], d_draft, d_bonus, d_ctx, out=so)
        ctx.verify_attn(st["q"], st["k"], st["v"], st["bt"], d_ctx, so.cu_q, cfg.t_cap, out=st["attn"])
        ctx.accept_into(st["logits"], d_draft, so.cu_q, cfg.t_cap, st["accept_len"], st["bonus"], st["toks"], st["total"])

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        step()                                                                   # warm-up outside capture
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            step()
    torch.cuda.synchronize()

    rng = np.random.default_rng(5)
    confs = [sel.conf, np.clip(sel.conf * rng.uniform(0.3, 1.2, sel.conf.shape), 0, 1).astype(np.float32),
             np.ones_like(sel.conf), np.zeros_like(sel.conf)]
    seen = set()
    for conf in confs:
        ref = orc.select(conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens, cost)
        T = ref.t_total
        seen.add(T)
        # the caller's part: pack the retained rows for the depths this input leads to (known here from the oracle)
        st["conf"].copy_(torch.from_numpy(conf))
        qp, lp = _pack_rows(cfg, ref.depths, q_all), _pack_rows(cfg, ref.depths, logits_all)
        st["q"][:T].copy_(qp)
        st["logits"][:T].copy_(lp)
        for _ in range(2):
            graph.replay()
        torch.cuda.synchronize()
        assert ctx.poll_device_status() == 0
        assert np.array_equal(so.depths.cpu().numpy(), ref.depths) and np.array_equal(so.cu_q.cpu().numpy(), ref.cu_q)
        ref_attn, _ = orc.verify_attn(qp, kv.k_cache, kv.v_cache, kv.block_table, sel.ctx_lens, ref.cu_q,
                                      cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
        ok, worst = attn_tolerance_ok(st["attn"][:T].float().cpu().numpy(), ref_attn)
        assert ok, f"worst err/limit {worst}"
        ra = orc.accept(lp, sel.draft_ids, ref.cu_q, cfg.gamma)
        assert np.array_equal(st["accept_len"].cpu().numpy(), ra.accept_len)
        assert np.array_equal(st["bonus"].cpu().numpy(), ra.bonus)
        assert np.array_equal(st["toks"].cpu().numpy(), ra.out_tokens) and int(st["total"].item()) == ra.n_accepted_total
    assert len(seen) >= 3                                                        # the one graph served different packed lengths
    ctx.close()


def test_work_list_from_the_selector_equals_the_attention_call_s_own():
    """Same batch through dcut_verify_attn with its own plan kernel and with the list the selector left: the same
    work list, hence bit-identical outputs; a call with other buffers falls back to its own plan."""
    cfg = wl.custom_config(B=20, gamma=16, n_q_heads=32, n_kv_heads=8, head_dim=128, ctx_lo=0, ctx_hi=1200)
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    cost = wl.cost_table_linear(cfg.t_cap + 1, 0.2, 0.002)
    ref = orc.select(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens, cost)
    q = dev(wl.q_rows(cfg, ref.depths))
    d_conf, d_draft, d_bonus, d_ctx = dev(sel.conf), dev(sel.draft_ids), dev(sel.bonus_ids), dev(sel.ctx_lens)
    d_k, d_v, d_bt = dev(kv.k_cache), dev(kv.v_cache), dev(kv.block_table)
    outs = []
    for on in (False, True):
        ctx = make_ctx(cfg, max_pages=kv.max_pages_per_req)
        ctx.set_cost_dense(cost)
        ctx.enable_plan_in_select(on)
        so = ctx.select(d_conf, d_draft, d_bonus, d_ctx)
        a = ctx.verify_attn(q, d_k, d_v, d_bt, d_ctx, so.cu_q, cfg.t_cap).clone()
        b = ctx.verify_attn(q, d_k, d_v, d_bt, d_ctx, so.cu_q, cfg.t_cap).clone()        # the list serves a second call
        # other buffers (a copy of cu_q): not the selector's batch as far as the library can tell -> own plan
        c = ctx.verify_attn(q, d_k, d_v, d_bt, d_ctx, so.cu_q.clone(), cfg.t_cap).clone()
        # and a different batch afterwards (full depth) must not see the stale list
        full = np.full(cfg.B, cfg.gamma, np.int32)
        qf = dev(wl.q_rows(cfg, full))
        d = ctx.verify_attn(qf, d_k, d_v, d_bt, d_ctx, dev(wl.cu_q_from_depths(full)), cfg.t_cap).clone()
        torch.cuda.synchronize()
        assert ctx.poll_device_status() == 0
        assert torch.equal(a, b) and torch.equal(a, c)
        outs.append((a, d))
        ctx.close()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    ref_attn, _ = orc.verify_attn(q.cpu(), kv.k_cache, kv.v_cache, kv.block_table, sel.ctx_lens, ref.cu_q,
                                  cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
    ok, worst = attn_tolerance_ok(outs[1][0].float().cpu().numpy(), ref_attn)
    assert ok, f"worst err/limit {worst}"
