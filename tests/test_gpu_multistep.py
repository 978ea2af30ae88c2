"""Several consecutive verify steps on the GPU (select -> verify_attn -> accept -> commit, no host round trip inside a
step) against the same chain of oracle calls: context lengths, next bonus tokens and the emitted token streams bit for
bit, attention within its tolerance at every step."""
import numpy as np
import pytest
import torch

from oracle import dcut_oracle as orc
from paper_2607_14647_b200 import workloads as wl
from tests.gpu_helpers import attn_tolerance_ok, dev, make_ctx

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,gamma,hq,hkv,dh", [(4, 16, 4, 1, 64), (6, 8, 8, 2, 128)])
def test_steps_chain(B, gamma, hq, hkv, dh):
    steps, V = 4, 300
    mk = lambda s: wl.custom_config(B=B, gamma=gamma, n_q_heads=hq, n_kv_heads=hkv, head_dim=dh, vocab=V, index=500 + s,
                                    ctx_lo=40, ctx_hi=120)
    cfg = mk(0)
    sel0 = wl.select_inputs(cfg)
    room = steps * (gamma + 1)
    kv = wl.paged_kv(cfg, sel0.ctx_lens + room)                 # pages for every step's appended tokens
    max_ctx = kv.max_pages_per_req * cfg.page_size
    cost = wl.cost_table_linear(cfg.t_cap + 1, 1.0, 0.05)
    ctx = make_ctx(cfg, max_pages=kv.max_pages_per_req, vocab=V)
    ctx.set_cost_dense(cost)
    d_k, d_v, d_bt = dev(kv.k_cache), dev(kv.v_cache), dev(kv.block_table)
    d_ctx, d_bonus = dev(sel0.ctx_lens.copy()), dev(sel0.bonus_ids.copy())
    cap_stream = steps * (gamma + 1)
    d_stream = torch.full((B, cap_stream), -1, dtype=torch.int32, device="cuda")
    d_slen = torch.zeros(B, dtype=torch.int32, device="cuda")
    ref_ctx, ref_bonus = sel0.ctx_lens.copy(), sel0.bonus_ids.copy()
    ref_streams = [[] for _ in range(B)]
    for s in range(steps):
        sel = wl.select_inputs(mk(s))
        draft = (sel.draft_ids % V).astype(np.int32)
        ref = orc.select(sel.conf, draft, ref_bonus, ref_ctx, cost)
        out = ctx.select(dev(sel.conf), dev(draft), d_bonus, d_ctx)
        torch.cuda.synchronize()
        assert np.array_equal(out.depths.cpu().numpy(), ref.depths)
        T = ref.t_total
        assert np.array_equal(out.tok_id.cpu().numpy()[:T], ref.tok_id) and np.array_equal(out.tok_pos.cpu().numpy()[:T], ref.tok_pos)
        q = wl.q_rows(mk(s), ref.depths)
        o = ctx.verify_attn(dev(q), d_k, d_v, d_bt, d_ctx, out.cu_q, cfg.t_cap)
        want, _ = orc.verify_attn(q, kv.k_cache, kv.v_cache, kv.block_table, ref_ctx, ref.cu_q, hq, hkv, dh, cfg.page_size)
        ok, worst = attn_tolerance_ok(o.float().cpu().numpy()[:T].reshape(want.shape), want)
        assert ok, worst
        sel_v = wl.SelectInputs(sel.conf, draft, sel.bonus_ids, sel.ctx_lens, sel.reject_index)
        logits = wl.logits_rows(mk(s), sel_v, ref.depths, vocab=V)
        al, bo, toks, total = ctx.accept(dev(logits), dev(draft), out.cu_q, cfg.t_cap)
        ctx.commit(al, toks, d_ctx, d_bonus, max_ctx, d_stream, d_slen)
        torch.cuda.synchronize()
        assert ctx.poll_device_status() == 0
        acc = orc.accept(logits, draft, ref.cu_q, gamma)
        ref_ctx, ref_bonus = orc.commit(acc.accept_len, acc.out_tokens, ref_ctx, ref_streams)
        assert np.array_equal(d_ctx.cpu().numpy(), ref_ctx) and np.array_equal(d_bonus.cpu().numpy(), ref_bonus)
    got_len = d_slen.cpu().numpy()
    got = d_stream.cpu().numpy()
    for i in range(B):
        assert got_len[i] == len(ref_streams[i]) and got[i, : got_len[i]].tolist() == ref_streams[i]
        assert (got[i, got_len[i]:] == -1).all()


def test_commit_reports_a_full_stream_and_a_full_context():
    cfg = wl.custom_config(B=2, gamma=4, vocab=10)
    ctx = make_ctx(cfg, vocab=10)
    al = dev(np.array([4, 0], np.int32))
    toks = dev(np.array([[1, 2, 3, 4, 5], [7, -1, -1, -1, -1]], np.int32))
    d_ctx, d_bonus = dev(np.array([10, 20], np.int32)), dev(np.zeros(2, np.int32))
    stream, slen = torch.full((2, 4), -1, dtype=torch.int32, device="cuda"), torch.zeros(2, dtype=torch.int32, device="cuda")
    ctx.commit(al, toks, d_ctx, d_bonus, 1000, stream, slen)         # request 0 needs 5 slots, the stream has 4
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 5
    assert slen.cpu().tolist() == [0, 1] and d_ctx.cpu().tolist() == [15, 21] and d_bonus.cpu().tolist() == [5, 7]
    ctx.commit(al, toks, d_ctx, d_bonus, 25, None, None)             # no room for the next block behind 20 + ...
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 5
    assert ctx.poll_device_status() == 0                             # polling clears the word
