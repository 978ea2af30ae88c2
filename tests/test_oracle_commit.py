"""Pins for the end-of-step bookkeeping (Section 3.1: a request commits its accepted drafts plus one token; Appendix A:
every request advances by at least one token per step)."""
import numpy as np

from oracle import dcut_oracle as orc
from paper_2607_14647_b200 import workloads as wl


def test_hand_example():
    # gamma = 3.  request 0 accepted 2 drafts then emitted 9; request 1 accepted none and emitted 4
    out_tokens = np.array([[5, 6, 9, -1], [4, -1, -1, -1]], np.int32)
    streams = [[1], []]
    ctx, nxt = orc.commit(np.array([2, 0]), out_tokens, np.array([100, 7]), streams)
    assert list(ctx) == [103, 8] and list(nxt) == [9, 4]
    assert streams == [[1, 5, 6, 9], [4]]


def test_three_steps_chain():
    cfg = wl.custom_config(B=5, gamma=6, vocab=50, index=400)
    cost = wl.cost_table_linear(cfg.t_cap + 1, 1.0, 0.05)
    ctx_lens = None
    streams = [[] for _ in range(cfg.B)]
    bonus = None
    emitted = 0
    for step in range(3):
        sel = wl.select_inputs(wl.custom_config(B=5, gamma=6, vocab=50, index=400 + step))
        if ctx_lens is None:
            ctx_lens, bonus = sel.ctx_lens.copy(), sel.bonus_ids.copy()
        ref = orc.select(sel.conf, sel.draft_ids, bonus, ctx_lens, cost)
        assert ref.tok_id[ref.cu_q[:-1]].tolist() == bonus.tolist()       # the previous closing token leads the block
        logits = wl.logits_rows(cfg, sel, ref.depths, vocab=50)
        acc = orc.accept(logits, sel.draft_ids % 50, ref.cu_q, cfg.gamma)
        before = ctx_lens.copy()
        ctx_lens, bonus = orc.commit(acc.accept_len, acc.out_tokens, ctx_lens, streams)
        assert np.array_equal(ctx_lens - before, acc.accept_len + 1) and (ctx_lens - before >= 1).all()
        assert np.array_equal(bonus, acc.bonus)
        emitted += acc.n_accepted_total
    assert sum(len(s) for s in streams) == emitted
    assert [s[-1] for s in streams] == bonus.tolist()
