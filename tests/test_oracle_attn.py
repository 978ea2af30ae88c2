"""Pins for the attention oracle: numpy float64 softmax written from the definition, and the
properties the definition implies (decode special case, causality, GQA, page invariance)."""
import numpy as np
import pytest
import torch

from oracle import dcut_oracle as orc
from paper_2607_14647_b200 import workloads as wl


def _setup(cfg, depths):
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    q = wl.q_rows(cfg, depths)
    return sel, kv, q, wl.cu_q_from_depths(depths)


def _numpy_attention(cfg, q, kv, ctx_lens, depths):
    """softmax(q k^T / sqrt(Dh)) v per request with a bottom-right-aligned causal mask,
    gathering each request's keys from its pages, all in float64."""
    K = kv.k_cache.double().numpy()
    V = kv.v_cache.double().numpy()
    Q = q.double().numpy()
    cu = wl.cu_q_from_depths(depths)
    out = np.zeros((int(cu[-1]), cfg.n_q_heads, cfg.head_dim))
    lse = np.zeros((int(cu[-1]), cfg.n_q_heads))
    for i, d in enumerate(depths):
        n = int(ctx_lens[i]) + int(d) + 1
        pages = kv.block_table[i, : (n + cfg.page_size - 1) // cfg.page_size]
        # [pages, Hkv, ps, Dh] -> [Hkv, tokens, Dh]
        Ki = K[pages].transpose(1, 0, 2, 3).reshape(cfg.n_kv_heads, -1, cfg.head_dim)[:, :n]
        Vi = V[pages].transpose(1, 0, 2, 3).reshape(cfg.n_kv_heads, -1, cfg.head_dim)[:, :n]
        Ki = np.repeat(Ki, cfg.group, axis=0)
        Vi = np.repeat(Vi, cfg.group, axis=0)
        Qi = Q[cu[i]: cu[i + 1]]                                    # [1+d, Hq, Dh]
        s = np.einsum("thd,hjd->htj", Qi, Ki) / np.sqrt(cfg.head_dim)
        t_idx = np.arange(d + 1)[:, None]
        j_idx = np.arange(n)[None, :]
        s = np.where(j_idx <= ctx_lens[i] + t_idx, s, -np.inf)
        m = s.max(-1, keepdims=True)
        e = np.exp(s - m)
        z = e.sum(-1, keepdims=True)
        out[cu[i]: cu[i + 1]] = np.einsum("htj,hjd->thd", e / z, Vi)
        lse[cu[i]: cu[i + 1]] = (m + np.log(z))[..., 0].T
    return out, lse


@pytest.mark.parametrize("depths", [[16, 16, 16, 16], [0, 3, 16, 7], [0, 0, 0, 0]])
def test_matches_numpy_float64_on_tiny_config(depths):
    cfg = wl.config(0)
    depths = np.array(depths, np.int32)
    sel, kv, q, cu = _setup(cfg, depths)
    out, lse = orc.verify_attn(q, kv.k_cache, kv.v_cache, kv.block_table, sel.ctx_lens, cu,
                               cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
    want, want_lse = _numpy_attention(cfg, q, kv, sel.ctx_lens, depths)
    np.testing.assert_allclose(out, want, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(lse, want_lse, rtol=1e-12, atol=1e-12)


def test_gqa_shape_matches_numpy():
    cfg = wl.custom_config(B=3, gamma=5, n_q_heads=8, n_kv_heads=2, head_dim=32, ctx_lo=5, ctx_hi=70)
    depths = np.array([5, 0, 2], np.int32)
    sel, kv, q, cu = _setup(cfg, depths)
    out, lse = orc.verify_attn(q, kv.k_cache, kv.v_cache, kv.block_table, sel.ctx_lens, cu,
                               cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
    want, want_lse = _numpy_attention(cfg, q, kv, sel.ctx_lens, depths)
    np.testing.assert_allclose(out, want, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(lse, want_lse, rtol=1e-12)


def test_depth_zero_is_plain_decode_attention():
    """d_i = 0: one query over the L_i cached tokens plus itself."""
    cfg = wl.config(0)
    depths = np.zeros(cfg.B, np.int32)
    sel, kv, q, cu = _setup(cfg, depths)
    out, _ = orc.verify_attn(q, kv.k_cache, kv.v_cache, kv.block_table, sel.ctx_lens, cu,
                             cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
    K, V = kv.k_cache.double().numpy(), kv.v_cache.double().numpy()
    for i in range(cfg.B):
        n = int(sel.ctx_lens[i]) + 1
        keys = np.stack([K[kv.block_table[i, j // 16], 0, j % 16] for j in range(n)])
        vals = np.stack([V[kv.block_table[i, j // 16], 0, j % 16] for j in range(n)])
        for h in range(cfg.n_q_heads):
            s = keys @ q[i, h].double().numpy() / 8.0
            w = np.exp(s - s.max())
            np.testing.assert_allclose(out[i, h], (w / w.sum()) @ vals, rtol=1e-11, atol=1e-12)


def test_equal_values_give_that_vector():
    cfg = wl.config(0)
    depths = np.array([4, 0, 9, 16], np.int32)
    sel, kv, q, cu = _setup(cfg, depths)
    vec = torch.randn(cfg.head_dim, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    v = kv.v_cache.clone()
    v[:] = vec
    out, _ = orc.verify_attn(q, kv.k_cache, v, kv.block_table, sel.ctx_lens, cu,
                             cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
    np.testing.assert_allclose(out, np.broadcast_to(vec.double().numpy(), out.shape), rtol=1e-12)


def test_causality():
    """Changing K/V at block position t' leaves tokens t < t' bit-unchanged and moves t >= t'."""
    cfg = wl.config(0)
    depths = np.full(cfg.B, 8, np.int32)
    sel, kv, q, cu = _setup(cfg, depths)
    args = (kv.block_table, sel.ctx_lens, cu, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
    base, _ = orc.verify_attn(q, kv.k_cache, kv.v_cache, *args)
    tp = 5
    k2, v2 = kv.k_cache.clone(), kv.v_cache.clone()
    for i in range(cfg.B):
        j = int(sel.ctx_lens[i]) + tp
        k2[kv.block_table[i, j // 16], :, j % 16] += 1.0
        v2[kv.block_table[i, j // 16], :, j % 16] += 1.0
    out, _ = orc.verify_attn(q, k2, v2, *args)
    for i in range(cfg.B):
        a = cu[i]
        assert np.array_equal(out[a: a + tp], base[a: a + tp])
        assert not np.allclose(out[a + tp: a + 9], base[a + tp: a + 9])
    # positions beyond the deepest query (slots L_i + d_i + 1 ...) are never read
    k3, v3 = kv.k_cache.clone(), kv.v_cache.clone()
    for i in range(cfg.B):
        for j in range(int(sel.ctx_lens[i]) + 9, int(sel.ctx_lens[i]) + 17):
            k3[kv.block_table[i, j // 16], :, j % 16] = 1.0e4
            v3[kv.block_table[i, j // 16], :, j % 16] = 1.0e4
    out3, _ = orc.verify_attn(q, k3, v3, *args)
    assert np.array_equal(out3, base)


def test_gqa_equal_queries_equal_outputs():
    cfg = wl.custom_config(B=2, gamma=4, n_q_heads=8, n_kv_heads=2, head_dim=32, ctx_lo=20, ctx_hi=40)
    depths = np.array([4, 2], np.int32)
    sel, kv, q, cu = _setup(cfg, depths)
    q = q.clone()
    q[:, 1:4] = q[:, 0:1]        # heads 0..3 share kv head 0
    out, _ = orc.verify_attn(q, kv.k_cache, kv.v_cache, kv.block_table, sel.ctx_lens, cu,
                             cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
    for h in (1, 2, 3):
        assert np.array_equal(out[:, h], out[:, 0])
    q[:, 4] = q[:, 0]            # head 4 reads kv head 1: same query, different keys
    out, _ = orc.verify_attn(q, kv.k_cache, kv.v_cache, kv.block_table, sel.ctx_lens, cu,
                             cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
    assert not np.allclose(out[:, 4], out[:, 0])


def test_physical_page_permutation_leaves_output_unchanged():
    cfg = wl.config(0)
    depths = np.array([2, 16, 0, 5], np.int32)
    sel, kv, q, cu = _setup(cfg, depths)
    args = (sel.ctx_lens, cu, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
    base, _ = orc.verify_attn(q, kv.k_cache, kv.v_cache, kv.block_table, *args)
    perm = np.random.default_rng(5).permutation(kv.num_pages)
    inv = np.argsort(perm)
    k2, v2 = kv.k_cache[torch.from_numpy(perm)], kv.v_cache[torch.from_numpy(perm)]   # new[p] = old[perm[p]]
    bt2 = np.where(kv.block_table >= 0, inv[np.maximum(kv.block_table, 0)], -1).astype(np.int32)
    out, _ = orc.verify_attn(q, k2, v2, bt2, *args)
    assert np.array_equal(out, base)


def test_sampled_rows_equal_full_rows():
    cfg = wl.config(0)
    depths = np.array([3, 16, 0, 8], np.int32)
    sel, kv, q, cu = _setup(cfg, depths)
    args = (q, kv.k_cache, kv.v_cache, kv.block_table, sel.ctx_lens, cu, cfg.n_q_heads, cfg.n_kv_heads,
            cfg.head_dim, cfg.page_size)
    full, lse = orc.verify_attn(*args)
    tok = np.array([0, 3, 4, 20, 21, 30], np.int32)
    head = np.array([0, 3, 1, 2, 0, 3], np.int32)
    part, lse_p = orc.verify_attn(*args, sample_tok=tok, sample_head=head)
    assert np.array_equal(part, full[tok, head]) and np.array_equal(lse_p, lse[tok, head])
