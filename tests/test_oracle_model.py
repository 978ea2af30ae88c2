"""Pins for the oracle's layer and whole-model compositions (`layer_forward`, `model_verify`).

The pieces (RMSNorm, linear, RoPE, SwiGLU, paged attention, acceptance) have their own pins; what is checked here is
the wiring between them: operand order, residuals, head layout of the fused QKV rows, GQA head mapping, positions,
the cache append, which cache a layer reads, the final norm, the row each request's prediction comes from.
  * a dense textbook decoder (contiguous per-request sequences, full causal score matrices, fp64, no paging, no
    intermediate rounding) written out below from the definition of the architecture;
  * the property the method rests on (Section 3.1): the retained prefix of a request is verified exactly as it
    would be without pruning, i.e. cutting a request's depth leaves the rows that remain unchanged;
  * requests are independent; identity layers reduce the model to embedding + norm + head.
"""
import numpy as np
import torch

from oracle import dcut_oracle as orc
from paper_2607_14647_b200 import workloads as wl

HQ, HKV, DH, PS = 4, 2, 32, 16
HID, INTER, VOCAB = 64, 96, 50
EPS, THETA = 1e-6, 1e4


def _cfg(B=3):
    return wl.custom_config(B=B, gamma=4, n_q_heads=HQ, n_kv_heads=HKV, head_dim=DH, ctx_lo=3, ctx_hi=40, vocab=VOCAB)


def _names(w):
    return {n: getattr(w, n) for n in ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")}


def _setup(n_layers, B=3, scale_w=4.0):
    cfg = _cfg(B)
    sel = wl.select_inputs(cfg)
    mw = wl.model_weights(cfg, n_layers, VOCAB, HID, INTER)
    layers = []
    for w in mw.layers:                       # larger weights than the 0.02 init so that every branch matters
        d = _names(w)
        for k in ("w_qkv", "w_o", "w_gate", "w_up", "w_down"):
            d[k] = (d[k].float() * scale_w).to(torch.bfloat16)
        layers.append(d)
    kvs = [wl.paged_kv(cfg, sel.ctx_lens, layer=l) for l in range(n_layers)]
    return cfg, sel, mw, layers, kvs


def _rms(x, g):
    return x / np.sqrt((x ** 2).mean(-1, keepdims=True) + EPS) * g


def _rope(x, pos):
    """x [n, heads, DH]; rotates the pair (e, e + DH/2) by pos * theta^(-2e/DH)."""
    half = DH // 2
    ang = pos[:, None, None] * THETA ** (-np.arange(half) / half)[None, None, :]
    z = (x[..., :half] + 1j * x[..., half:]) * np.exp(1j * ang)
    return np.concatenate([z.real, z.imag], -1)


def _dense_layer(x_rows, w, kc, vc, bt, L, d):
    """One request: x_rows [d+1, HID] are the new tokens at positions L .. L+d; cached K/V come from the pages."""
    W = {k: v.double().numpy() for k, v in w.items()}
    pos_new = np.arange(L, L + d + 1).astype(np.float64)
    n = _rms(x_rows, W["g_attn"])
    qkv = n @ W["w_qkv"].T
    q = _rope(qkv[:, : HQ * DH].reshape(-1, HQ, DH), pos_new)
    k_new = _rope(qkv[:, HQ * DH: (HQ + HKV) * DH].reshape(-1, HKV, DH), pos_new)
    v_new = qkv[:, (HQ + HKV) * DH:].reshape(-1, HKV, DH)
    k_old = np.stack([kc[bt[p // PS], :, p % PS].double().numpy() for p in range(L)]) if L else np.zeros((0, HKV, DH))
    v_old = np.stack([vc[bt[p // PS], :, p % PS].double().numpy() for p in range(L)]) if L else np.zeros((0, HKV, DH))
    K, V = np.concatenate([k_old, k_new]), np.concatenate([v_old, v_new])
    a = np.empty((d + 1, HQ, DH))
    for h in range(HQ):
        g = h // (HQ // HKV)
        s = q[:, h] @ K[:, g].T / np.sqrt(DH)
        for t in range(d + 1):
            s[t, L + t + 1:] = -np.inf                                   # token t sees the context and tokens <= t
        p = np.exp(s - s.max(-1, keepdims=True))
        a[:, h] = (p / p.sum(-1, keepdims=True)) @ V[:, g]
    h1 = x_rows + a.reshape(d + 1, HQ * DH) @ W["w_o"].T
    n2 = _rms(h1, W["g_mlp"])
    gate, up = n2 @ W["w_gate"].T, n2 @ W["w_up"].T
    return h1 + (gate / (1 + np.exp(-gate)) * up) @ W["w_down"].T


def _dense_model(tok, mw, layers, kvs, bt, ctx_lens, depths):
    cu = wl.cu_q_from_depths(depths)
    x = mw.embed.double().numpy()[tok]
    for l, w in enumerate(layers):
        y = np.empty_like(x)
        for i, d in enumerate(depths):
            y[cu[i]:cu[i + 1]] = _dense_layer(x[cu[i]:cu[i + 1]], w, kvs[l].k_cache, kvs[l].v_cache, bt[i],
                                              int(ctx_lens[i]), int(d))
        x = y
    return x, _rms(x, mw.g_final.double().numpy()) @ mw.w_lm.double().numpy().T


def _oracle_model(tok, mw, layers, kvs, sel, depths):
    return orc.model_verify(tok, mw.embed, layers, mw.g_final, mw.w_lm, [k.k_cache for k in kvs],
                            [k.v_cache for k in kvs], kvs[0].block_table if kvs else np.zeros((len(depths), 1), np.int32),
                            sel.ctx_lens, depths, sel.draft_ids % VOCAB, HQ, HKV, DH, PS, EPS, THETA)


def test_one_layer_against_the_dense_textbook_decoder():
    cfg, sel, mw, layers, kvs = _setup(1)
    depths = np.array([4, 0, 2], np.int32)
    x = wl.layer_x_rows(cfg, depths, HID)
    st = orc.layer_forward(x, layers[0], kvs[0].k_cache, kvs[0].v_cache, kvs[0].block_table, sel.ctx_lens, depths,
                           HQ, HKV, DH, PS, EPS, THETA)
    cu = wl.cu_q_from_depths(depths)
    xd = x.double().numpy()
    want = np.concatenate([_dense_layer(xd[cu[i]:cu[i + 1]], layers[0], kvs[0].k_cache, kvs[0].v_cache,
                                        kvs[0].block_table[i], int(sel.ctx_lens[i]), int(d)) for i, d in enumerate(depths)])
    got = st["y"].double().numpy()
    # nine tensors are rounded to bf16 on the way (2^-9 relative each); the branches add to an output of size ~ |x|
    assert np.abs(got - want).max() <= 0.03 * np.abs(want).max()
    assert np.abs(got - want).mean() <= 0.004 * np.abs(want).mean()
    # a wrong wiring moves the output by far more than the rounding: e.g. dropping the attention branch
    no_attn = dict(layers[0], w_o=torch.zeros_like(layers[0]["w_o"]))
    other = np.concatenate([_dense_layer(xd[cu[i]:cu[i + 1]], no_attn, kvs[0].k_cache, kvs[0].v_cache, kvs[0].block_table[i],
                                         int(sel.ctx_lens[i]), int(d)) for i, d in enumerate(depths)])
    assert np.abs(other - want).mean() > 0.1 * np.abs(want).mean()


def test_two_layer_model_against_the_dense_textbook_decoder():
    cfg, sel, mw, layers, kvs = _setup(2)
    depths = np.array([3, 4, 0], np.int32)
    tok = wl.model_tok_ids(sel, depths, VOCAB)
    res, logits, hidden, caches = _oracle_model(tok, mw, layers, kvs, sel, depths)
    x_want, logits_want = _dense_model(tok, mw, layers, kvs, kvs[0].block_table, sel.ctx_lens, depths)
    assert np.abs(hidden[1].double().numpy() - x_want).mean() <= 0.006 * np.abs(x_want).mean()
    assert np.abs(logits - logits_want).max() <= 0.03 * np.abs(logits_want).max()
    # layer 1 must read ITS cache: the dense model given layer 0's cache twice lands elsewhere
    _, wrong = _dense_model(tok, mw, layers, [kvs[0], kvs[0]], kvs[0].block_table, sel.ctx_lens, depths)
    assert np.abs(wrong - logits_want).mean() > 10 * np.abs(logits - logits_want).mean()
    # acceptance follows the logits the oracle itself reports
    cu = wl.cu_q_from_depths(depths)
    am = orc._as_bf16_tensor(orc.round_bf16(logits)).float().numpy().argmax(1)      # first index among equal values
    for i, d in enumerate(depths):
        m = 0
        while m < d and am[cu[i] + m] == sel.draft_ids[i, m] % VOCAB:
            m += 1
        assert res.accept_len[i] == m and res.bonus[i] == am[cu[i] + m]
    # the caches returned hold the new tokens of every layer at positions L_i + t, nothing else changed
    for l in range(2):
        changed = (caches[l][0] != kvs[l].k_cache).any(-1).any(1)          # [pages, slots]
        want_changed = torch.zeros_like(changed)
        for i, d in enumerate(depths):
            for t in range(d + 1):
                p = int(sel.ctx_lens[i]) + t
                want_changed[kvs[l].block_table[i, p // PS], p % PS] = True
        assert torch.equal(changed, want_changed)


def _model_with_drafts(tok_of, draft_ids, mw, layers, kvs, sel, depths):
    return orc.model_verify(tok_of(depths), mw.embed, layers, mw.g_final, mw.w_lm, [k.k_cache for k in kvs],
                            [k.v_cache for k in kvs], kvs[0].block_table, sel.ctx_lens, depths, draft_ids,
                            HQ, HKV, DH, PS, EPS, THETA)


def test_cutting_a_request_leaves_its_retained_rows_unchanged():
    cfg, sel, mw, layers, kvs = _setup(2)
    gamma, B = 4, 3
    deep = np.full(B, gamma, np.int32)
    bonus0 = sel.bonus_ids % VOCAB
    drafts = np.zeros((B, gamma), np.int64)

    def tok_of(depths):
        return np.concatenate([np.concatenate([[bonus0[i]], drafts[i, : int(d)]]) for i, d in enumerate(depths)])

    # drafts that the target itself would produce (greedy decoding with the oracle, one more position per pass) ...
    cu = wl.cu_q_from_depths(deep)
    for t in range(gamma):
        _, logits, _, _ = _model_with_drafts(tok_of, drafts, mw, layers, kvs, sel, deep)
        am = orc._as_bf16_tensor(orc.round_bf16(logits)).float().numpy().argmax(1)
        drafts[:, t] = am[cu[:-1] + t]
    # ... then spoiled at position 2 for request 1 and position 1 for request 2: accepted lengths 4, 2, 1
    drafts[1, 2] = (drafts[1, 2] + 1) % VOCAB
    drafts[2, 1] = (drafts[2, 1] + 1) % VOCAB
    a = _model_with_drafts(tok_of, drafts, mw, layers, kvs, sel, deep)
    assert list(a[0].accept_len) == [4, 2, 1]
    for cut in (np.array([4, 1, 0], np.int32), np.array([2, 3, 1], np.int32), np.array([0, 0, 4], np.int32)):
        b = _model_with_drafts(tok_of, drafts, mw, layers, kvs, sel, cut)
        cub = wl.cu_q_from_depths(cut)
        for i in range(B):
            assert np.array_equal(a[1][cu[i]: cu[i] + cut[i] + 1], b[1][cub[i]:cub[i + 1]])   # logits of the retained rows
            # accepted length under the cut = min(uncut accepted length, depth): Section 3.1's truncation
            assert b[0].accept_len[i] == min(a[0].accept_len[i], cut[i])
            assert b[0].bonus[i] == am_row(a[1], cu[i] + b[0].accept_len[i])


def am_row(logits, r):
    return int(orc._as_bf16_tensor(orc.round_bf16(logits[r:r + 1])).float().numpy().argmax(1)[0])


def test_requests_are_independent_and_identity_layers_vanish():
    cfg, sel, mw, layers, kvs = _setup(2)
    depths = np.array([2, 3, 1], np.int32)
    tok = wl.model_tok_ids(sel, depths, VOCAB)
    base = _oracle_model(tok, mw, layers, kvs, sel, depths)
    tok2 = tok.copy()
    tok2[0] = (tok2[0] + 1) % VOCAB                                         # first token of request 0
    other = _oracle_model(tok2, mw, layers, kvs, sel, depths)
    cu = wl.cu_q_from_depths(depths)
    assert np.array_equal(base[1][cu[1]:], other[1][cu[1]:]) and not np.array_equal(base[1][:cu[1]], other[1][:cu[1]])
    ident = [dict(w, w_o=torch.zeros_like(w["w_o"]), w_down=torch.zeros_like(w["w_down"])) for w in layers]
    r_id = _oracle_model(tok, mw, ident, kvs, sel, depths)
    r_0 = _oracle_model(tok, mw, [], [], sel, depths)
    assert np.array_equal(r_id[1], r_0[1]) and np.array_equal(r_id[0].accept_len, r_0[0].accept_len)
    want = _rms(mw.embed.double().numpy()[tok], mw.g_final.double().numpy())
    assert np.abs(r_0[2][-1].double().numpy() - want).max() <= 2.0 ** -8 * np.abs(want).max()
