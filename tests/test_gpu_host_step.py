"""dcut_verify_step_host (the whole step from host buffers: copies in, select, attention, acceptance, copies out)
against the oracle: depths, accepted lengths, bonus and emitted tokens bit-exact, the attention output of the retained
rows within 1e-2 + 1e-2 |ref|, and the byte counts it reports against the tensors it has to move."""
import numpy as np
import pytest
import torch

from oracle import dcut_oracle as orc
from paper_2607_14647_b200 import workloads as wl
from tests.gpu_helpers import attn_tolerance_ok, dev, make_ctx

pytestmark = pytest.mark.gpu


def _case(cfg, cost):
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    full = np.full(cfg.B, cfg.gamma, np.int32)
    q_all = wl.q_rows(cfg, full).view(cfg.B, cfg.gamma + 1, cfg.n_q_heads, cfg.head_dim).contiguous()
    logits_all = wl.logits_rows(cfg, sel, full).view(cfg.B, cfg.gamma + 1, cfg.vocab).contiguous()
    ctx = make_ctx(cfg, max_pages=kv.max_pages_per_req)
    ctx.set_cost_dense(cost)
    d_k, d_v = dev(kv.k_cache), dev(kv.v_cache)
    t = torch.from_numpy
    outs = []
    for _ in range(2):                       # the second call reuses the context's staging buffers and streams
        out = ctx.verify_step_host(t(sel.conf), t(sel.draft_ids), t(sel.bonus_ids), t(sel.ctx_lens), t(kv.block_table),
                                   q_all, logits_all, d_k, d_v, want_attn_out=True)
        assert ctx.poll_device_status() == 0
        outs.append({k: (v.clone() if isinstance(v, torch.Tensor) else v) for k, v in out.items()})
    ctx.close()
    for k in ("depths", "accept_len", "bonus", "out_tokens", "n_accepted_total", "attn_out"):
        assert torch.equal(outs[0][k], outs[1][k])
    out = outs[0]
    ref = orc.select(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens, cost)
    depths = out["depths"].numpy()
    assert np.array_equal(depths, ref.depths)
    cu = wl.cu_q_from_depths(depths)
    T = int(cu[-1])
    rows = np.concatenate([i * (cfg.gamma + 1) + np.arange(d + 1) for i, d in enumerate(depths)])
    q = q_all.view(-1, cfg.n_q_heads, cfg.head_dim)[rows].contiguous()
    lg = logits_all.view(-1, cfg.vocab)[rows].contiguous()
    acc = orc.accept(lg, sel.draft_ids, cu, cfg.gamma)
    assert np.array_equal(out["accept_len"].numpy(), acc.accept_len) and np.array_equal(out["bonus"].numpy(), acc.bonus)
    assert np.array_equal(out["out_tokens"].numpy(), acc.out_tokens) and int(out["n_accepted_total"]) == acc.n_accepted_total
    ref_o, _ = orc.verify_attn(q, kv.k_cache, kv.v_cache, kv.block_table, sel.ctx_lens, cu, cfg.n_q_heads, cfg.n_kv_heads,
                               cfg.head_dim, cfg.page_size)
    ok, worst = attn_tolerance_ok(out["attn_out"][:T].float().numpy(), ref_o)
    assert ok, f"worst err/limit {worst}"
    row_bytes = cfg.n_q_heads * cfg.head_dim * 2 + cfg.vocab * 2
    want_h2d = sel.conf.nbytes + sel.draft_ids.nbytes + sel.bonus_ids.nbytes + sel.ctx_lens.nbytes + kv.block_table.nbytes + T * row_bytes
    assert out["h2d_bytes"] == want_h2d                      # only the retained rows of Q and of the logits travel
    assert out["d2h_bytes"] == 4 * (cfg.B + 1 + 3 * cfg.B + cfg.B * (cfg.gamma + 1) + 1) + T * cfg.n_q_heads * cfg.head_dim * 2


def test_tiny_config():
    cfg = wl.config(0)
    _case(cfg, wl.cost_table_for(cfg))


def test_mid_size_pruned_and_full_depth():
    cfg = wl.custom_config(B=12, gamma=16, n_q_heads=16, n_kv_heads=4, head_dim=128, ctx_lo=10, ctx_hi=700, vocab=4000)
    _case(cfg, wl.cost_table_linear(cfg.t_cap + 1, 0.2, 0.004))       # prunes
    _case(cfg, np.ones(cfg.t_cap + 1, np.float32))                    # flat cost: every draft is kept


def test_hidden_state_form_ends_in_the_lm_head():
    """dcut_verify_step_host given last hidden states + a resident LM head instead of logits rows: same selection and
    attention, acceptance through dcut_lm_head_accept.  Accepted lengths against the oracle's LM head + acceptance
    (the planted accepts win by a wide margin); every output equal to the device-side call on the same packed rows;
    the bytes that cross the bus counted from the hidden rows, not from logits."""
    cfg = wl.custom_config(B=10, gamma=8, n_q_heads=8, n_kv_heads=2, head_dim=128, ctx_lo=10, ctx_hi=500, vocab=1000, index=77)
    H = 512
    sel = wl.select_inputs(cfg)
    draft = (sel.draft_ids % cfg.vocab).astype(np.int32)
    sel_v = wl.SelectInputs(sel.conf, draft, sel.bonus_ids, sel.ctx_lens, sel.reject_index)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    cost = wl.cost_table_linear(cfg.t_cap + 1, 0.2, 0.004)
    full = np.full(cfg.B, cfg.gamma, np.int32)
    q_all = wl.q_rows(cfg, full).view(cfg.B, cfg.gamma + 1, cfg.n_q_heads, cfg.head_dim).contiguous()
    w_lm = wl.lm_head_weight(cfg, vocab=cfg.vocab, hidden=H)
    x_all = wl.lm_head_x_rows(cfg, sel_v, full, w_lm).view(cfg.B, cfg.gamma + 1, H).contiguous()
    ctx = make_ctx(cfg, max_pages=kv.max_pages_per_req, hidden=H, intermediate=H)
    ctx.set_cost_dense(cost)
    t = torch.from_numpy
    d_w = dev(w_lm)
    out = ctx.verify_step_host(t(sel.conf), t(draft), t(sel.bonus_ids), t(sel.ctx_lens), t(kv.block_table), q_all, None,
                               dev(kv.k_cache), dev(kv.v_cache), hidden_rows=x_all, w_lm=d_w)
    assert ctx.poll_device_status() == 0
    ref = orc.select(sel.conf, draft, sel.bonus_ids, sel.ctx_lens, cost)
    depths = out["depths"].numpy()
    assert np.array_equal(depths, ref.depths)
    cu = wl.cu_q_from_depths(depths)
    T = int(cu[-1])
    rows = np.concatenate([i * (cfg.gamma + 1) + np.arange(d + 1) for i, d in enumerate(depths)])
    xp = x_all.view(-1, H)[rows].contiguous()
    ref_acc, _ = orc.lm_head_accept(xp, w_lm, draft, cu, cfg.gamma)
    assert np.array_equal(out["accept_len"].numpy(), ref_acc.accept_len)
    assert np.array_equal(out["accept_len"].numpy(), np.minimum(sel.reject_index, depths))
    assert (out["bonus"].numpy() == ref_acc.bonus).mean() >= 0.9
    # the device-side call on the same packed rows gives the same outputs bit for bit
    xd = torch.zeros((cfg.t_cap, H), dtype=torch.bfloat16, device="cuda")
    xd[:T] = dev(xp)
    al, bo, toks, total, _ = ctx.lm_head_accept(xd, d_w, dev(draft), dev(cu), cfg.t_cap, row_argmax=True)
    torch.cuda.synchronize()
    assert np.array_equal(out["accept_len"].numpy(), al.cpu().numpy()) and np.array_equal(out["bonus"].numpy(), bo.cpu().numpy())
    assert np.array_equal(out["out_tokens"].numpy(), toks.cpu().numpy()) and int(out["n_accepted_total"]) == int(total.item())
    row_bytes = cfg.n_q_heads * cfg.head_dim * 2 + H * 2
    want_h2d = sel.conf.nbytes + draft.nbytes + sel.bonus_ids.nbytes + sel.ctx_lens.nbytes + kv.block_table.nbytes + T * row_bytes
    assert out["h2d_bytes"] == want_h2d
    ctx.close()
