"""Shared set-up of the GPU parity tests: upload seeded inputs, run the oracle beside the CUDA path."""
import numpy as np
import torch

from oracle import dcut_oracle as orc
from paper_2607_14647_b200 import workloads as wl


def dev(a, dtype=None):
    if isinstance(a, np.ndarray):
        a = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        a = a.to(dtype)
    return a.contiguous().cuda()


def make_ctx(cfg, max_pages=0, **kw):
    from paper_2607_14647_b200 import binding
    args = dict(max_B=cfg.B, max_gamma=cfg.gamma, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
                head_dim=cfg.head_dim, page_size=cfg.page_size, max_pages_per_req=max(max_pages, 1), vocab=cfg.vocab)
    args.update(kw)
    return binding.Context(**args)


def select_both(ctx, sel, cost=None, bucket=None, want=True):
    """Runs dcut_select and the oracle on the same inputs; returns (gpu SelectOut, oracle SelectResult)."""
    B, g = sel.conf.shape
    if bucket is not None:
        K, c = bucket
        ctx.set_cost_buckets(B, g, K, c)
        ref = orc.select(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens, np.asarray(c, np.float32), bucket_K=K)
    else:
        ctx.set_cost_dense(cost)
        ref = orc.select(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens, cost)
    out = ctx.select(dev(sel.conf), dev(sel.draft_ids), dev(sel.bonus_ids), dev(sel.ctx_lens),
                     want_scores=want, want_ranks=want)
    torch.cuda.synchronize()
    return out, ref


def assert_select_equal(out, ref):
    from paper_2607_14647_b200 import binding
    info = binding.read_info(out.info)
    assert info.n_star == ref.n_star and info.t_total == ref.t_total and info.candidate == ref.candidate
    assert info.sum_fixed == ref.sum_fixed
    assert np.float64(info.objective).tobytes() == np.float64(ref.objective).tobytes()
    assert np.array_equal(out.depths.cpu().numpy(), ref.depths)
    assert np.array_equal(out.cu_q.cpu().numpy(), ref.cu_q)
    T = ref.t_total
    for got, want in ((out.tok_req, ref.tok_req), (out.tok_pos, ref.tok_pos), (out.tok_id, ref.tok_id)):
        g = got.cpu().numpy()
        assert np.array_equal(g[:T], want) and np.all(g[T:] == -1)
    if out.scores is not None:
        assert out.scores.cpu().numpy().tobytes() == ref.scores.tobytes()
    if out.ranks is not None:
        assert np.array_equal(out.ranks.cpu().numpy(), ref.ranks)


def attn_tolerance_ok(got, want):
    """|err| <= 1e-2 + 1e-2 * |ref| (bf16 in, fp32 accumulate)."""
    got = np.asarray(got, np.float64)
    err = np.abs(got - want)
    lim = 1e-2 + 1e-2 * np.abs(want)
    return bool((err <= lim).all()), float((err / lim).max())
