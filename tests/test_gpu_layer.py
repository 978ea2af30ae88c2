"""Decoder-layer path against the oracle: the tcgen05 GEMM by itself (all three epilogues), RMSNorm + RoPE + cache
append through the whole layer on a small shape (every element, every stage that is visible), and the full-layer
workload on a sub-batch of requests the oracle can afford.  Tolerance 2e-2 + 2e-2 |ref| (bf16 tensors, fp32
accumulation over K up to 12 288; the paper gives none); for the layer output, |ref| is the larger of the output and of
the residual stream h1 it is added to, since both terms of that sum are rounded to bf16 before it."""
import numpy as np
import pytest
import torch

from oracle import dcut_oracle as orc
from paper_2607_14647_b200 import workloads as wl
from tests.gpu_helpers import dev, make_ctx

pytestmark = pytest.mark.gpu


def _f64(t):
    return t.float().cpu().numpy().astype(np.float64) if isinstance(t, torch.Tensor) else np.asarray(t, np.float64)


def _close(got, want, what, size=None):
    """|got - want| <= 2e-2 + 2e-2 s elementwise, s = |want|, or the larger of |want| and |size| where the value is a
    sum whose terms were rounded to bf16 on their own (the layer output y = h1 + MLP: an element that is 1.24 after
    attention and 0.10 after the MLP carries the rounding step of 1.24)."""
    got, want = _f64(got), _f64(want)
    err = np.abs(got - want)
    lim = 2e-2 + 2e-2 * (np.abs(want) if size is None else np.maximum(np.abs(want), np.abs(_f64(size))))
    assert (err <= lim).all(), f"{what}: worst err/limit {(err / lim).max():.2f} at {np.unravel_index((err / lim).argmax(), err.shape)}"


def _bf(rng, shape, scale=1.0):
    return torch.from_numpy((rng.standard_normal(shape, dtype=np.float32) * scale)).to(torch.bfloat16)


@pytest.mark.parametrize("T,N,K", [(1, 256, 64), (100, 256, 128), (128, 512, 512), (129, 256, 1024), (300, 768, 4096),
                                   (517, 256, 12288)])
def test_gemm_plain_and_residual(T, N, K):
    rng = np.random.default_rng(T + N + K)
    cfg = wl.custom_config(B=1, gamma=16, n_q_heads=4, n_kv_heads=2, head_dim=128)
    ctx = make_ctx(cfg, max_pages=1, vocab=0)
    T_cap = max(T, 2)
    a, w, res = _bf(rng, (T_cap, K)), _bf(rng, (N, K), 0.05), _bf(rng, (T_cap, N))
    cu = dev(np.array([0, T], np.int32))
    out = torch.full((T_cap, N), 7.0, dtype=torch.bfloat16, device="cuda")
    ctx.gemm_bf16(dev(a), dev(w), cu, T_cap, out)
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    ref = orc.linear(a[:T], w)
    _close(out[:T], ref, "plain")
    assert (out[T:] == 7.0).all()                      # rows past T are never stored
    out2 = torch.empty((T_cap, N), dtype=torch.bfloat16, device="cuda")
    ctx.gemm_bf16(dev(a), dev(w), cu, T_cap, out2, mode=1, residual=dev(res))
    _close(out2[:T], ref + res[:T].double().numpy(), "residual")
    ctx.close()


@pytest.mark.parametrize("T,I,K", [(70, 128, 256), (260, 384, 512), (131, 1024, 4096)])
def test_gemm_swiglu(T, I, K):
    rng = np.random.default_rng(T + I + K)
    cfg = wl.custom_config(B=1, gamma=16, n_q_heads=4, n_kv_heads=2, head_dim=128)
    ctx = make_ctx(cfg, max_pages=1, vocab=0)
    a, wg, wu = _bf(rng, (T, K)), _bf(rng, (I, K), 0.05), _bf(rng, (I, K), 0.05)
    out = torch.empty((T, I), dtype=torch.bfloat16, device="cuda")
    ctx.gemm_bf16(dev(a), dev(wg), dev(np.array([0, T], np.int32)), T, out, mode=2, w2=dev(wu))
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    _close(out, orc.swiglu_f64(orc.linear(a, wg), orc.linear(a, wu)), "swiglu")
    ctx.close()


def _layer_case(cfg, depths, hidden, inter, sub=None):
    """Runs the GPU layer on the whole batch and the oracle on the requests in `sub` (default: all)."""
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    w = wl.layer_weights(cfg, hidden, inter)
    wd = {n: getattr(w, n) for n in ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")}
    x = wl.layer_x_rows(cfg, depths, hidden)
    cu = wl.cu_q_from_depths(depths)
    tok_req = np.concatenate([np.full(d + 1, i) for i, d in enumerate(depths)]).astype(np.int32)
    tok_pos = np.concatenate([sel.ctx_lens[i] + np.arange(d + 1) for i, d in enumerate(depths)]).astype(np.int32)
    ctx = make_ctx(cfg, max_pages=kv.max_pages_per_req, hidden=hidden, intermediate=inter, vocab=0)
    d_k, d_v = dev(kv.k_cache), dev(kv.v_cache)
    y = torch.empty((int(cu[-1]), hidden), dtype=torch.bfloat16, device="cuda")
    ctx.layer_forward({k: dev(v) for k, v in wd.items()}, dev(x), y, d_k, d_v, dev(kv.block_table), dev(sel.ctx_lens),
                      dev(cu), dev(tok_req), dev(tok_pos), cfg.t_cap, cfg.rms_eps, cfg.rope_theta)
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    ctx.close()
    sub = list(range(cfg.B)) if sub is None else sub
    rows = np.concatenate([np.arange(cu[i], cu[i + 1]) for i in sub])
    ref = orc.layer_forward(x[rows], wd, kv.k_cache, kv.v_cache, kv.block_table[sub], sel.ctx_lens[sub], depths[sub],
                            cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.page_size, cfg.rms_eps, cfg.rope_theta)
    _close(y[rows], ref["y"], "layer output y", size=ref["h1"])
    # the appended K/V of the new tokens (the rest of the cache must be untouched)
    kc, vc = d_k.cpu(), d_v.cpu()
    for n_, i in enumerate(sub):
        for t in range(depths[i] + 1):
            pos = int(sel.ctx_lens[i]) + t
            page = kv.block_table[i, pos // 16]
            _close(kc[page, :, pos % 16], ref["k_cache"][page, :, pos % 16], "appended K")
            _close(vc[page, :, pos % 16], ref["v_cache"][page, :, pos % 16], "appended V")
    if len(sub) == cfg.B:
        touched = torch.zeros(kc.shape[0], dtype=torch.bool)
        for i in range(cfg.B):
            for t in range(depths[i] + 1):
                touched[kv.block_table[i, (int(sel.ctx_lens[i]) + t) // 16]] = True
        assert torch.equal(kc[~touched], kv.k_cache[~touched]) and torch.equal(vc[~touched], kv.v_cache[~touched])


def test_small_layer_every_element():
    cfg = wl.custom_config(B=6, gamma=16, n_q_heads=4, n_kv_heads=2, head_dim=128, ctx_lo=5, ctx_hi=400,
                           conf_kind="skew_halves")
    _layer_case(cfg, np.array([16, 0, 3, 9, 1, 16], np.int32), hidden=512, inter=1024)


def test_full_layer_workload_on_sampled_requests():
    cfg = wl.config(4)
    sel = wl.select_inputs(cfg)
    depths = orc.select(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens,
                        wl.cost_table_linear(cfg.t_cap + 1, 0.5, 0.001)).depths
    _layer_case(cfg, depths, cfg.hidden, cfg.intermediate, sub=[0, 1, 37])


@pytest.mark.parametrize("arm", ["full_gamma", "T512"])
def test_full_layer_workload_at_the_bench_s_packed_lengths(arm):
    """The two packed lengths the benchmark times on the layer workload: T = 1088 (full depth: the length at which the
    GEMM plan picks pair tiles for the wide projections) and T = 512 (the pruned arm: the selector forced to the
    budget the profiled table leads to), through dcut_layer_forward at the full shapes, on three sampled requests."""
    cfg = wl.config(4)
    sel = wl.select_inputs(cfg)
    if arm == "full_gamma":
        depths = np.full(cfg.B, cfg.gamma, np.int32)
    else:
        depths = orc.select(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens, np.ones(1, np.float32), bucket_K=[512]).depths
        assert int(depths.sum()) + cfg.B == 512
    deep = int(np.argmax(depths))
    _layer_case(cfg, depths, cfg.hidden, cfg.intermediate, sub=[2, deep, 61])


@pytest.mark.parametrize("T,N,K,mode", [(300, 512, 1024, 0), (257, 256, 4096, 1), (640, 1024, 512, 2), (100, 256, 128, 0)])
def test_single_sm_mode_matches_the_oracle(T, N, K, mode, monkeypatch):
    """The GEMM with its pair mode (cta_group::2) switched off when the context is created: single-SM tiles only.
    (The default build picks the mode per launch; the other GEMM tests cover that.)"""
    monkeypatch.setenv("DCUT_GEMM_2CTA", "0")
    rng = np.random.default_rng(T + N + K + mode)
    cfg = wl.custom_config(B=1, gamma=16, n_q_heads=4, n_kv_heads=2, head_dim=128)
    ctx = make_ctx(cfg, max_pages=1, vocab=0)
    T_cap = T + 5
    a, w = _bf(rng, (T_cap, K)), _bf(rng, (N, K), 0.05)
    w2 = _bf(rng, (N, K), 0.05) if mode == 2 else None
    res = _bf(rng, (T_cap, N)) if mode == 1 else None
    cu = dev(np.array([0, T], np.int32))
    out = torch.full((T_cap, N), 7.0, dtype=torch.bfloat16, device="cuda")
    ctx.gemm_bf16(dev(a), dev(w), cu, T_cap, out, mode=mode, w2=None if w2 is None else dev(w2),
                  residual=None if res is None else dev(res))
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    if mode == 2:
        want = orc.swiglu_f64(orc.linear(a[:T], w), orc.linear(a[:T], w2))
    else:
        want = orc.linear(a[:T], w) + (res[:T].double().numpy() if mode == 1 else 0.0)
    _close(out[:T], want, f"single-SM mode, epilogue {mode}")
    assert (out[T:].float() == 7.0).all()       # rows past T are never written


@pytest.mark.parametrize("T,N,K,mode", [(300, 512, 8192, 0), (257, 256, 8192, 1), (640, 1024, 8192, 2), (40, 256, 8192, 0)])
def test_pair_mode_matches_the_oracle(T, N, K, mode):
    """Shapes for which the kernel picks its pair mode (one wave either way and K >= 8192), every stored epilogue."""
    rng = np.random.default_rng(T + N + K + mode)
    cfg = wl.custom_config(B=1, gamma=16, n_q_heads=4, n_kv_heads=2, head_dim=128)
    ctx = make_ctx(cfg, max_pages=1, vocab=0)
    T_cap = T + 5
    a, w = _bf(rng, (T_cap, K)), _bf(rng, (N, K), 0.05)
    w2 = _bf(rng, (N, K), 0.05) if mode == 2 else None
    res = _bf(rng, (T_cap, N)) if mode == 1 else None
    cu = dev(np.array([0, T], np.int32))
    out = torch.full((T_cap, N), 7.0, dtype=torch.bfloat16, device="cuda")
    ctx.gemm_bf16(dev(a), dev(w), cu, T_cap, out, mode=mode, w2=None if w2 is None else dev(w2),
                  residual=None if res is None else dev(res))
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    if mode == 2:
        want = orc.swiglu_f64(orc.linear(a[:T], w), orc.linear(a[:T], w2))
    else:
        want = orc.linear(a[:T], w) + (res[:T].double().numpy() if mode == 1 else 0.0)
    _close(out[:T], want, f"pair mode, epilogue {mode}")
    assert (out[T:].float() == 7.0).all()       # rows past T are never written


@pytest.mark.parametrize("width_bit", [1, 2, 3, 4, 5, 6])
@pytest.mark.parametrize("mode", [0, 1, 2])
def test_every_tile_width_matches_the_oracle(width_bit, mode, monkeypatch):
    """The one-SM mode picks its tile width (256, 224, ..., 64 columns) per launch; with only one narrower width allowed
    and less than a wave of tiles the narrower one is always the cheaper.  N = 768 is not a multiple of most widths
    (ragged last tile: zero-filled weight rows, masked stores); T spans three row blocks with a ragged last one."""
    if mode == 2 and width_bit % 2:
        pytest.skip("the SwiGLU tile uses the widths whose halves are multiples of 32 columns")
    monkeypatch.setenv("DCUT_GEMM_WIDTHS", str(1 | (1 << width_bit)))
    T, N, K = 300, 768, 512
    rng = np.random.default_rng(100 * width_bit + mode)
    cfg = wl.custom_config(B=1, gamma=16, n_q_heads=4, n_kv_heads=2, head_dim=128)
    ctx = make_ctx(cfg, max_pages=1, vocab=0)
    T_cap = T + 3
    a, w = _bf(rng, (T_cap, K)), _bf(rng, (N, K), 0.05)
    w2 = _bf(rng, (N, K), 0.05) if mode == 2 else None
    res = _bf(rng, (T_cap, N)) if mode == 1 else None
    out = torch.full((T_cap, N), 7.0, dtype=torch.bfloat16, device="cuda")
    ctx.gemm_bf16(dev(a), dev(w), dev(np.array([0, T], np.int32)), T_cap, out, mode=mode, w2=None if w2 is None else dev(w2),
                  residual=None if res is None else dev(res))
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    if mode == 2:
        want = orc.swiglu_f64(orc.linear(a[:T], w), orc.linear(a[:T], w2))
    else:
        want = orc.linear(a[:T], w) + (res[:T].double().numpy() if mode == 1 else 0.0)
    _close(out[:T], want, f"width bit {width_bit}, epilogue {mode}")
    assert (out[T:].float() == 7.0).all()
    ctx.close()


@pytest.mark.parametrize("width_bit", [1, 2, 4, 6])
@pytest.mark.parametrize("mode", [0, 1, 2])
def test_pair_mode_at_every_tile_width(width_bit, mode, monkeypatch):
    """The pair mode (two SMs per 256-row tile) with a narrower tile, forced through the experiment knob; ragged last
    column tile and ragged last row block as above."""
    monkeypatch.setenv("DCUT_GEMM_FORCE", str(8 + width_bit))
    T, N, K = 300, 768, 8192
    rng = np.random.default_rng(1000 + 100 * width_bit + mode)
    cfg = wl.custom_config(B=1, gamma=16, n_q_heads=4, n_kv_heads=2, head_dim=128)
    ctx = make_ctx(cfg, max_pages=1, vocab=0)
    T_cap = T + 3
    a, w = _bf(rng, (T_cap, K), 0.5), _bf(rng, (N, K), 0.05)
    w2 = _bf(rng, (N, K), 0.05) if mode == 2 else None
    res = _bf(rng, (T_cap, N)) if mode == 1 else None
    out = torch.full((T_cap, N), 7.0, dtype=torch.bfloat16, device="cuda")
    ctx.gemm_bf16(dev(a), dev(w), dev(np.array([0, T], np.int32)), T_cap, out, mode=mode, w2=None if w2 is None else dev(w2),
                  residual=None if res is None else dev(res))
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    if mode == 2:
        want = orc.swiglu_f64(orc.linear(a[:T], w), orc.linear(a[:T], w2))
    else:
        want = orc.linear(a[:T], w) + (res[:T].double().numpy() if mode == 1 else 0.0)
    _close(out[:T], want, f"pair mode, width bit {width_bit}, epilogue {mode}")
    assert (out[T:].float() == 7.0).all()
    ctx.close()


@pytest.mark.parametrize("width_bit", [0, 1, 3, 4, 6])
@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("T,K", [(300, 1024), (120, 192), (257, 12288)])
def test_split_k_mode_at_every_tile_width(width_bit, mode, T, K, monkeypatch):
    """Both SMs of a pair on one 128-row tile, half of the k-blocks each (an odd count too: K = 192 is three), partial
    sums exchanged through distributed shared memory; forced through the experiment knob.  N = 768 keeps the tiles
    within one wave of pairs and leaves a ragged last column tile for most widths."""
    monkeypatch.setenv("DCUT_GEMM_FORCE", str(16 + width_bit))
    N = 768
    rng = np.random.default_rng(2000 + 100 * width_bit + mode + T)
    cfg = wl.custom_config(B=1, gamma=16, n_q_heads=4, n_kv_heads=2, head_dim=128)
    ctx = make_ctx(cfg, max_pages=1, vocab=0)
    T_cap = T + 3
    a, w = _bf(rng, (T_cap, K), 0.5), _bf(rng, (N, K), 0.05)
    res = _bf(rng, (T_cap, N)) if mode == 1 else None
    out = torch.full((T_cap, N), 7.0, dtype=torch.bfloat16, device="cuda")
    ctx.gemm_bf16(dev(a), dev(w), dev(np.array([0, T], np.int32)), T_cap, out, mode=mode,
                  residual=None if res is None else dev(res))
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    want = orc.linear(a[:T], w) + (res[:T].double().numpy() if mode == 1 else 0.0)
    _close(out[:T], want, f"split-K, width bit {width_bit}, epilogue {mode}")
    assert (out[T:].float() == 7.0).all()
    ctx.close()


def test_first_layer_call_captured_in_a_graph_replays_correctly():
    """The first layer call on a context uploads the RoPE frequency table from host memory.  Captured into a CUDA
    graph, that upload is a node that runs again at every replay, so its source must outlive the call (it lives in
    the context): two replays of a graph whose capture was the context's very first call equal the eager result."""
    cfg = wl.custom_config(B=5, gamma=16, n_q_heads=4, n_kv_heads=2, head_dim=128, ctx_lo=5, ctx_hi=300, conf_kind="skew_halves")
    hidden, inter = 512, 1024
    depths = np.array([16, 0, 3, 9, 1], np.int32)
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    w = wl.layer_weights(cfg, hidden, inter)
    wd = {n: dev(getattr(w, n)) for n in ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")}
    x = dev(wl.layer_x_rows(cfg, depths, hidden))
    cu = dev(wl.cu_q_from_depths(depths))
    tok_req = dev(np.concatenate([np.full(d + 1, i) for i, d in enumerate(depths)]).astype(np.int32))
    tok_pos = dev(np.concatenate([sel.ctx_lens[i] + np.arange(d + 1) for i, d in enumerate(depths)]).astype(np.int32))
    d_bt, d_ctx = dev(kv.block_table), dev(sel.ctx_lens)

    def run(ctx, y, k, v):
        ctx.layer_forward(wd, x, y, k, v, d_bt, d_ctx, cu, tok_req, tok_pos, cfg.t_cap, cfg.rms_eps, cfg.rope_theta)

    eager_ctx = make_ctx(cfg, max_pages=kv.max_pages_per_req, hidden=hidden, intermediate=inter, vocab=0)
    y_eager = torch.empty((int(depths.sum()) + cfg.B, hidden), dtype=torch.bfloat16, device="cuda")
    k_e, v_e = dev(kv.k_cache), dev(kv.v_cache)
    run(eager_ctx, y_eager, k_e, v_e)
    torch.cuda.synchronize()
    eager_ctx.close()

    ctx = make_ctx(cfg, max_pages=kv.max_pages_per_req, hidden=hidden, intermediate=inter, vocab=0)
    y = torch.zeros_like(y_eager)
    k_g, v_g = dev(kv.k_cache), dev(kv.v_cache)
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            run(ctx, y, k_g, v_g)                      # the context's first layer call happens inside the capture
    torch.cuda.synchronize()
    for _ in range(2):
        y.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert ctx.poll_device_status() == 0
        assert torch.equal(y, y_eager) and torch.equal(k_g, k_e) and torch.equal(v_g, v_e)
    ctx.close()


@pytest.mark.parametrize("tp", [2, 4])
def test_tensor_parallel_halves_reproduce_the_layer(tp):
    """dcut_layer_attn_part / dcut_layer_mlp_part / dcut_residual_add: the decoder layer cut where a tensor-parallel
    deployment exchanges.  Rank r holds the q / k / v heads, O columns, gate / up rows and down columns of its share
    and its slice of the paged cache; the ranks run one after the other on this one GPU and a float32 sum stands in
    for the two all-reduces (the exchange is the caller's).  The result must match the oracle's layer like the
    unsharded call does, and the appended K/V slices must be the unsharded call's (same arithmetic per head)."""
    cfg = wl.custom_config(B=6, gamma=16, n_q_heads=8, n_kv_heads=4, head_dim=128, ctx_lo=5, ctx_hi=400, conf_kind="skew_halves")
    hidden, inter = 512, 1024
    depths = np.array([16, 0, 3, 9, 1, 16], np.int32)
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    w = wl.layer_weights(cfg, hidden, inter)
    wd = {n: getattr(w, n) for n in ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")}
    x = wl.layer_x_rows(cfg, depths, hidden)
    cu = wl.cu_q_from_depths(depths)
    T = int(cu[-1])
    tok_req = np.concatenate([np.full(d + 1, i) for i, d in enumerate(depths)]).astype(np.int32)
    tok_pos = np.concatenate([sel.ctx_lens[i] + np.arange(d + 1) for i, d in enumerate(depths)]).astype(np.int32)
    d_x, d_cu, d_bt, d_ctx = dev(x), dev(cu), dev(kv.block_table), dev(sel.ctx_lens)
    d_req, d_pos = dev(tok_req), dev(tok_pos)
    Dh, Hq, Hkv = cfg.head_dim, cfg.n_q_heads, cfg.n_kv_heads
    hq, hk, it = Hq // tp, Hkv // tp, inter // tp
    shard_cfg = wl.custom_config(B=cfg.B, gamma=cfg.gamma, n_q_heads=hq, n_kv_heads=hk, head_dim=Dh, ctx_lo=cfg.ctx_lo, ctx_hi=cfg.ctx_hi)
    ranks = []
    for r in range(tp):
        q_rows = wd["w_qkv"][r * hq * Dh:(r + 1) * hq * Dh]
        k_rows = wd["w_qkv"][Hq * Dh + r * hk * Dh: Hq * Dh + (r + 1) * hk * Dh]
        v_rows = wd["w_qkv"][(Hq + Hkv) * Dh + r * hk * Dh: (Hq + Hkv) * Dh + (r + 1) * hk * Dh]
        ws = dict(w_qkv=torch.cat([q_rows, k_rows, v_rows]).contiguous(), w_o=wd["w_o"][:, r * hq * Dh:(r + 1) * hq * Dh].contiguous(),
                  w_gate=wd["w_gate"][r * it:(r + 1) * it].contiguous(), w_up=wd["w_up"][r * it:(r + 1) * it].contiguous(),
                  w_down=wd["w_down"][:, r * it:(r + 1) * it].contiguous(), g_attn=wd["g_attn"], g_mlp=wd["g_mlp"])
        ranks.append(dict(ctx=make_ctx(shard_cfg, max_pages=kv.max_pages_per_req, hidden=hidden, intermediate=it, vocab=0),
                          w={k: dev(v) for k, v in ws.items()},
                          k=dev(kv.k_cache[:, r * hk:(r + 1) * hk].contiguous()), v=dev(kv.v_cache[:, r * hk:(r + 1) * hk].contiguous())))
    bf = dict(dtype=torch.bfloat16, device="cuda")
    # attention half on every rank, then the first all-reduce
    parts = []
    for rk in ranks:
        o = torch.empty((T, hidden), **bf)
        rk["ctx"].layer_attn_part(rk["w"], d_x, o, rk["k"], rk["v"], d_bt, d_ctx, d_cu, d_req, d_pos, cfg.t_cap, cfg.rms_eps, cfg.rope_theta)
        parts.append(o)
    o_sum = torch.stack([p.float() for p in parts]).sum(0).to(torch.bfloat16)
    ys = []
    for rk in ranks:                                       # every rank computes h1 and its MLP half from the same sum
        h1 = rk["ctx"].residual_add(d_x, o_sum, torch.empty((T, hidden), **bf), d_cu, cfg.t_cap)
        rk["h1"] = h1
        rk["d"] = rk["ctx"].layer_mlp_part(rk["w"], h1, torch.empty((T, hidden), **bf), d_cu, cfg.t_cap, cfg.rms_eps, cfg.rope_theta)
    d_sum = torch.stack([rk["d"].float() for rk in ranks]).sum(0).to(torch.bfloat16)
    for rk in ranks:
        ys.append(rk["ctx"].residual_add(rk["h1"], d_sum, torch.empty((T, hidden), **bf), d_cu, cfg.t_cap))
    torch.cuda.synchronize()
    for rk in ranks:
        assert rk["ctx"].poll_device_status() == 0
    assert all(torch.equal(ys[0], y) for y in ys[1:])
    ref = orc.layer_forward(x, wd, kv.k_cache, kv.v_cache, kv.block_table, sel.ctx_lens, depths, Hq, Hkv, Dh, cfg.page_size,
                            cfg.rms_eps, cfg.rope_theta)
    _close(ys[0], ref["y"], "tensor-parallel layer output y", size=ref["h1"])
    # the unsharded call on the same inputs: same output within the layer's tolerance, same appended K/V bit for bit
    ctx = make_ctx(cfg, max_pages=kv.max_pages_per_req, hidden=hidden, intermediate=inter, vocab=0)
    y_full = torch.empty((T, hidden), **bf)
    k_full, v_full = dev(kv.k_cache), dev(kv.v_cache)
    ctx.layer_forward({k: dev(v) for k, v in wd.items()}, d_x, y_full, k_full, v_full, d_bt, d_ctx, d_cu, d_req, d_pos, cfg.t_cap,
                      cfg.rms_eps, cfg.rope_theta)
    torch.cuda.synchronize()
    _close(ys[0], y_full.float().cpu(), "tensor-parallel against unsharded")
    for r, rk in enumerate(ranks):
        assert torch.equal(rk["k"], k_full[:, r * hk:(r + 1) * hk]) and torch.equal(rk["v"], v_full[:, r * hk:(r + 1) * hk])
        rk["ctx"].close()
    ctx.close()
