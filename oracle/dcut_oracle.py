"""ctypes front end of the CPU oracle (`dcut_oracle.c`).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this module.
It marshals numpy / torch-CPU arrays to the C functions (what each C function computes, and the passage
of the paper it follows, is in the C file).  A few definitions that are only bookkeeping around those
functions are written out here in plain Python, each citing its passage: `commit` (end of a step),
`cost_grid_*` (the start-up cost table), and the compositions `lm_head_accept`, `layer_forward`,
`model_verify`.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dcut_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the library is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-Wall", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Info(C.Structure):
    _fields_ = [("n_star", C.c_int32), ("t_total", C.c_int32), ("candidate", C.c_int32),
                ("closure_ok", C.c_int32), ("sum_fixed", C.c_int64), ("objective", C.c_double),
                ("sum_f64", C.c_double)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
    return _lib


def _p(a, typ):
    if a is None:
        return None
    return a.ctypes.data_as(C.POINTER(typ))


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _bf16_bits(t) -> np.ndarray:
    """A torch bf16 CPU tensor (or a uint16 array of bf16 bit patterns) as contiguous uint16."""
    if isinstance(t, np.ndarray):
        assert t.dtype == np.uint16
        return np.ascontiguousarray(t)
    import torch
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def scores(conf: np.ndarray) -> np.ndarray:
    conf = np.ascontiguousarray(conf, dtype=np.float32)
    B, g = conf.shape
    out = np.empty((B, g), dtype=np.float32)
    rc = lib().oracle_scores(_p(conf, C.c_float), B, g, _p(out, C.c_float))
    assert rc == 0, rc
    return out


def budget(B: int, gamma: int, num: int, den: int) -> int:
    k = C.c_int(0)
    rc = lib().oracle_budget(B, gamma, num, den, C.byref(k))
    if rc != 0:
        raise ValueError(f"oracle_budget rc={rc}")
    return k.value


@dataclass
class SelectResult:
    depths: np.ndarray
    cu_q: np.ndarray
    tok_req: np.ndarray
    tok_pos: np.ndarray
    tok_id: np.ndarray
    ranks: np.ndarray      # [B, gamma] global rank of every draft position
    scores: np.ndarray     # [B, gamma] fp32
    n_star: int
    t_total: int
    candidate: int
    closure_ok: bool
    sum_fixed: int
    objective: float
    sum_f64: float


class OracleError(RuntimeError):
    def __init__(self, rc):
        super().__init__(f"oracle rc={rc}")
        self.rc = rc


def select(conf, draft_ids, bonus_ids, ctx_lens, cost_ms, bucket_K: Optional[Sequence[int]] = None) -> SelectResult:
    """Dense mode when bucket_K is None (cost_ms indexed by packed length T), else bucket mode
    (cost_ms per bucket)."""
    conf = np.ascontiguousarray(conf, dtype=np.float32)
    B, g = conf.shape
    draft_ids, bonus_ids, ctx_lens = _i32(draft_ids).reshape(B, g), _i32(bonus_ids), _i32(ctx_lens)
    cost_ms = np.ascontiguousarray(cost_ms, dtype=np.float32)
    cap = B * (g + 1)
    depths = np.zeros(B, np.int32)
    cu_q = np.zeros(B + 1, np.int32)
    tok_req = np.full(max(cap, 1), -1, np.int32)
    tok_pos = np.full(max(cap, 1), -1, np.int32)
    tok_id = np.full(max(cap, 1), -1, np.int32)
    ranks = np.zeros((B, g), np.int32)
    sc = np.zeros((B, g), np.float32)
    info = _Info()
    bk = None if bucket_K is None else _i32(bucket_K)
    rc = lib().oracle_select(_p(conf, C.c_float), B, g, _p(draft_ids, C.c_int32), _p(bonus_ids, C.c_int32),
                             _p(ctx_lens, C.c_int32), 0 if bk is None else 1, _p(cost_ms, C.c_float),
                             len(cost_ms), _p(bk, C.c_int32), _p(depths, C.c_int32), _p(cu_q, C.c_int32),
                             _p(tok_req, C.c_int32), _p(tok_pos, C.c_int32), _p(tok_id, C.c_int32),
                             _p(ranks, C.c_int32), _p(sc, C.c_float), C.byref(info))
    if rc != 0:
        raise OracleError(rc)
    T = info.t_total
    return SelectResult(depths, cu_q, tok_req[:T], tok_pos[:T], tok_id[:T], ranks, sc, info.n_star, T,
                        info.candidate, bool(info.closure_ok), info.sum_fixed, info.objective, info.sum_f64)


def commit(accept_len, out_tokens, ctx_lens, streams):
    """End of a step (Section 3.1): request i has emitted out_tokens[i, 0..m_i]; its context grows by m_i + 1 (the old
    bonus token and the m_i accepted drafts are now part of it), the closing token becomes the next bonus token, and the
    emitted tokens are appended to the request's stream (a list of lists, changed in place).
    Returns (new ctx_lens, next bonus_ids)."""
    accept_len, out_tokens, ctx_lens = _i32(accept_len), _i32(out_tokens), _i32(ctx_lens)
    new_ctx, nxt = ctx_lens.copy(), np.zeros(len(ctx_lens), np.int32)
    for i, m in enumerate(accept_len):
        new_ctx[i] = ctx_lens[i] + m + 1
        nxt[i] = out_tokens[i, m]
        streams[i].extend(int(t) for t in out_tokens[i, : m + 1])
    return new_ctx, nxt


# ---------------------------------------------------------------------------------------------
# Start-up cost table C(B, rho)  (Appendix C, "Cost-table profiling protocol"; Eq. 4; Table 3)

def cost_grid_median(samples_ms) -> np.float32:
    """"Median per-step latency over a small number of repetitions": the middle sample; for an even count the
    mean of the two middle samples (a reading: the paper does not say), in double, rounded once to fp32."""
    v = sorted(float(np.float32(x)) for x in samples_ms)
    n = len(v)
    return np.float32(v[n // 2]) if n % 2 else np.float32((v[n // 2 - 1] + v[n // 2]) * 0.5)


def cost_grid_nearest(batch_sizes: Sequence[int], B: int) -> int:
    """"Batch sizes that fall between captured points reuse the nearest captured entry": index of the captured
    size with the smallest |B_c - B|.  A tie (the paper is silent) goes to the larger captured batch."""
    best = None
    for b, bc in enumerate(batch_sizes):
        d = abs(int(bc) - int(B))
        if best is None or d < best[0] or (d == best[0] and bc > batch_sizes[best[1]]):
            best = (d, b)
    return best[1]


def cost_grid_buckets(batch_sizes, ratios, gamma: int, table, B: int):
    """The bucket table a live batch of B requests reads: budgets K_rho(B) by Eq. 4 for the live B, latencies from
    the row of the nearest captured batch size.  Ratios whose budgets coincide (small B) are one candidate; it
    keeps the smaller latency (a reading: the objective of Eq. 5 then prefers it anyway)."""
    row = table[cost_grid_nearest(batch_sizes, B)]
    out = {}
    for (num, den), c in zip(ratios, row):
        K = budget(B, gamma, num, den)
        out[K] = min(out.get(K, np.inf), float(np.float32(c)))
    Ks = sorted(out)
    return np.array(Ks, np.int32), np.array([out[k] for k in Ks], np.float32)


def scores_shifted(conf: np.ndarray) -> np.ndarray:
    """Eq. 7: the admission score of depth k is the product of the confidences before k."""
    conf = np.ascontiguousarray(conf, dtype=np.float32)
    B, g = conf.shape
    out = np.empty((B, g), dtype=np.float32)
    rc = lib().oracle_scores_shifted(_p(conf, C.c_float), B, g, _p(out, C.c_float))
    assert rc == 0, rc
    return out


def select_causal(conf, draft_ids, bonus_ids, ctx_lens, cost_ms) -> SelectResult:
    """Causal early-stopping frontier scan on the shifted scores (dense cost table); `ranks` is not filled."""
    conf = np.ascontiguousarray(conf, dtype=np.float32)
    B, g = conf.shape
    draft_ids, bonus_ids, ctx_lens = _i32(draft_ids).reshape(B, g), _i32(bonus_ids), _i32(ctx_lens)
    cost_ms = np.ascontiguousarray(cost_ms, dtype=np.float32)
    cap = B * (g + 1)
    depths = np.zeros(B, np.int32)
    cu_q = np.zeros(B + 1, np.int32)
    tok_req = np.full(max(cap, 1), -1, np.int32)
    tok_pos = np.full(max(cap, 1), -1, np.int32)
    tok_id = np.full(max(cap, 1), -1, np.int32)
    sc = np.zeros((B, g), np.float32)
    info = _Info()
    rc = lib().oracle_select_causal(_p(conf, C.c_float), B, g, _p(draft_ids, C.c_int32), _p(bonus_ids, C.c_int32),
                                    _p(ctx_lens, C.c_int32), _p(cost_ms, C.c_float), len(cost_ms),
                                    _p(depths, C.c_int32), _p(cu_q, C.c_int32), _p(tok_req, C.c_int32),
                                    _p(tok_pos, C.c_int32), _p(tok_id, C.c_int32), _p(sc, C.c_float), C.byref(info))
    if rc != 0:
        raise OracleError(rc)
    T = info.t_total
    return SelectResult(depths, cu_q, tok_req[:T], tok_pos[:T], tok_id[:T], np.zeros((B, g), np.int32), sc, info.n_star,
                        T, info.candidate, bool(info.closure_ok), info.sum_fixed, info.objective, info.sum_f64)


@dataclass
class AcceptRsResult:
    accept_len: np.ndarray
    bonus: np.ndarray
    out_tokens: np.ndarray
    n_accepted_total: int
    prob: np.ndarray       # [B, 2]: p(z)/q(z) of the deciding draft, residual mass (0 if fully accepted)


def accept_rs(target_logits, draft_logits, draft_ids, cu_q, gamma: int, u_accept, u_sample) -> AcceptRsResult:
    """Rejection-sampling acceptance; target_logits bf16 [T, V], draft_logits bf16 [B, gamma, V], u_accept fp32
    [B, gamma], u_sample fp32 [B]."""
    tb, db = _bf16_bits(target_logits), _bf16_bits(draft_logits)
    T, V = tb.shape
    cu_q = _i32(cu_q)
    B = len(cu_q) - 1
    assert int(cu_q[B]) <= T and db.size == B * gamma * V
    draft_ids = _i32(draft_ids).reshape(B, gamma)
    ua = np.ascontiguousarray(u_accept, dtype=np.float32).reshape(B, gamma)
    us = np.ascontiguousarray(u_sample, dtype=np.float32).reshape(B)
    al, bo = np.zeros(B, np.int32), np.zeros(B, np.int32)
    ot = np.zeros((B, gamma + 1), np.int32)
    tot = C.c_int32(0)
    prob = np.zeros((B, 2), np.float64)
    f = lib().oracle_accept_rs
    f.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_int] + [C.c_void_p] * 7
    rc = f(tb.ctypes.data, db.ctypes.data, V, draft_ids.ctypes.data, cu_q.ctypes.data, B, gamma, ua.ctypes.data,
           us.ctypes.data, al.ctypes.data, bo.ctypes.data, ot.ctypes.data, C.addressof(tot), prob.ctypes.data)
    if rc != 0:
        raise OracleError(rc)
    return AcceptRsResult(al, bo, ot, tot.value, prob)


def verify_attn(q, k_cache, v_cache, block_table, ctx_lens, cu_q, n_q_heads, n_kv_heads, head_dim,
                page_size, scale=None, sample_tok=None, sample_head=None):
    """Returns (out, lse) in float64: [T, Hq, Dh], [T, Hq], or [n, Dh], [n] for sampled rows."""
    qb, kb, vb = _bf16_bits(q), _bf16_bits(k_cache), _bf16_bits(v_cache)
    bt = _i32(block_table)
    B = bt.shape[0]
    ctx_lens, cu_q = _i32(ctx_lens), _i32(cu_q)
    T = int(cu_q[B])
    if scale is None:
        scale = 1.0 / np.sqrt(head_dim)
    if sample_tok is not None:
        st, sh = _i32(sample_tok), _i32(sample_head)
        n = len(st)
        out = np.empty((n, head_dim), np.float64)
        lse = np.empty((n,), np.float64)
    else:
        st = sh = None
        n = 0
        out = np.empty((T, n_q_heads, head_dim), np.float64)
        lse = np.empty((T, n_q_heads), np.float64)
    f = lib().oracle_verify_attn
    f.argtypes = [C.c_void_p] * 6 + [C.c_int] * 6 + [C.c_double, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p,
                                                     C.c_void_p]
    rc = f(qb.ctypes.data, kb.ctypes.data, vb.ctypes.data, bt.ctypes.data, ctx_lens.ctypes.data,
           cu_q.ctypes.data, B, n_q_heads, n_kv_heads, head_dim, page_size, bt.shape[1], float(scale),
           None if st is None else st.ctypes.data, None if sh is None else sh.ctypes.data, n,
           out.ctypes.data, lse.ctypes.data)
    if rc != 0:
        raise OracleError(rc)
    return out, lse


@dataclass
class AcceptResult:
    accept_len: np.ndarray
    bonus: np.ndarray
    out_tokens: np.ndarray
    n_accepted_total: int
    argmax: np.ndarray


def accept(logits, draft_ids, cu_q, gamma: int) -> AcceptResult:
    lb = _bf16_bits(logits)
    T, V = lb.shape
    cu_q = _i32(cu_q)
    B = len(cu_q) - 1
    assert int(cu_q[B]) <= T
    draft_ids = _i32(draft_ids).reshape(B, gamma)
    al = np.zeros(B, np.int32)
    bo = np.zeros(B, np.int32)
    ot = np.zeros((B, gamma + 1), np.int32)
    tot = C.c_int32(0)
    am = np.zeros(max(int(cu_q[B]), 1), np.int32)
    f = lib().oracle_accept
    f.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_int] + [C.c_void_p] * 5
    rc = f(lb.ctypes.data, V, draft_ids.ctypes.data, cu_q.ctypes.data, B, gamma, al.ctypes.data,
           bo.ctypes.data, ot.ctypes.data, C.addressof(tot), am.ctypes.data)
    if rc != 0:
        raise OracleError(rc)
    return AcceptResult(al, bo, ot, tot.value, am[: int(cu_q[B])])


# ---- decoder-layer pieces ---------------------------------------------------------------------

def round_bf16(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, np.uint16)
    f = lib().oracle_round_bf16
    f.argtypes = [C.c_void_p, C.c_long, C.c_void_p]
    f.restype = None
    f(x.ctypes.data, x.size, out.ctypes.data)
    return out


def rmsnorm(x, gain, eps: float) -> np.ndarray:
    xb, gb = _bf16_bits(x), _bf16_bits(gain)
    rows, hidden = xb.shape
    y = np.empty((rows, hidden), np.float64)
    f = lib().oracle_rmsnorm
    f.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_double, C.c_void_p]
    assert f(xb.ctypes.data, gb.ctypes.data, rows, hidden, float(eps), y.ctypes.data) == 0
    return y


def linear(a, w) -> np.ndarray:
    ab, wb = _bf16_bits(a), _bf16_bits(w)
    M, K = ab.shape
    N, K2 = wb.shape
    assert K == K2
    c = np.empty((M, N), np.float64)
    f = lib().oracle_linear
    f.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p]
    assert f(ab.ctypes.data, wb.ctypes.data, M, N, K, c.ctypes.data) == 0
    return c


def lm_head_accept(x, w_lm, draft_ids, cu_q, gamma: int):
    """The LM head followed by greedy acceptance (Section 3.1: the target's prediction at every retained position):
    logits = x . w_lm^T in fp64 from the bf16 inputs, rounded to bf16 (the tensor a target model hands to the
    acceptance step), then `accept`.  Returns (AcceptResult, logits fp64 [T, V])."""
    logits64 = linear(x, w_lm)
    res = accept(_as_bf16_tensor(round_bf16(logits64)), draft_ids, cu_q, gamma)
    return res, logits64


def rope(x, pos, theta: float) -> np.ndarray:
    xb = _bf16_bits(x)
    rows, heads, dh = xb.shape
    pos = _i32(pos)
    y = np.empty((rows, heads, dh), np.float64)
    f = lib().oracle_rope
    f.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_double, C.c_void_p]
    assert f(xb.ctypes.data, pos.ctypes.data, rows, heads, dh, float(theta), y.ctypes.data) == 0
    return y


def swiglu(g, u) -> np.ndarray:
    gb, ub = _bf16_bits(g), _bf16_bits(u)
    y = np.empty(gb.shape, np.float64)
    f = lib().oracle_swiglu
    f.argtypes = [C.c_void_p, C.c_void_p, C.c_long, C.c_void_p]
    assert f(gb.ctypes.data, ub.ctypes.data, gb.size, y.ctypes.data) == 0
    return y


def swiglu_f64(g: np.ndarray, u: np.ndarray) -> np.ndarray:
    g = np.ascontiguousarray(g, np.float64)
    u = np.ascontiguousarray(u, np.float64)
    y = np.empty(g.shape, np.float64)
    f = lib().oracle_swiglu_f64
    f.argtypes = [C.c_void_p, C.c_void_p, C.c_long, C.c_void_p]
    assert f(g.ctypes.data, u.ctypes.data, g.size, y.ctypes.data) == 0
    return y


def _as_bf16_tensor(bits: np.ndarray):
    import torch
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16)


def layer_forward(x, w, k_cache, v_cache, block_table, ctx_lens, depths, n_q_heads, n_kv_heads, head_dim, page_size,
                  rms_eps, rope_theta):
    """One pre-norm decoder layer on the packed batch, composed from the C pieces in double precision and
    rounded to bf16 exactly where the GPU path materialises a tensor: n, qkv, q/k after RoPE, attention
    output, h1, n2, the SwiGLU product, y.  `w` has w_qkv, w_o, w_gate, w_up, w_down, g_attn, g_mlp (torch bf16).
    The K/V of the new tokens are written into COPIES of the caches at positions L_i + t.  Returns a dict of the
    stages (torch bf16) plus the updated cache copies."""
    import torch
    depths = np.asarray(depths, np.int32)
    B = len(depths)
    cu = np.zeros(B + 1, np.int32)
    np.cumsum(depths.astype(np.int64) + 1, out=cu[1:])
    T = int(cu[-1])
    pos = np.concatenate([int(ctx_lens[i]) + np.arange(depths[i] + 1) for i in range(B)]).astype(np.int32)
    req = np.concatenate([np.full(depths[i] + 1, i) for i in range(B)])
    rb = lambda a: _as_bf16_tensor(round_bf16(a))
    n = rb(rmsnorm(x, w["g_attn"], rms_eps))
    qkv = rb(linear(n, w["w_qkv"]))
    q_w, kv_w = n_q_heads * head_dim, n_kv_heads * head_dim
    q = rb(rope(qkv[:, :q_w].reshape(T, n_q_heads, head_dim).contiguous(), pos, rope_theta))
    k = rb(rope(qkv[:, q_w:q_w + kv_w].reshape(T, n_kv_heads, head_dim).contiguous(), pos, rope_theta))
    v = qkv[:, q_w + kv_w:].reshape(T, n_kv_heads, head_dim)
    kc, vc = k_cache.clone(), v_cache.clone()
    for r in range(T):
        page = int(block_table[req[r], pos[r] // page_size])
        kc[page, :, pos[r] % page_size] = k[r]
        vc[page, :, pos[r] % page_size] = v[r]
    attn, _ = verify_attn(q, kc, vc, block_table, ctx_lens, cu, n_q_heads, n_kv_heads, head_dim, page_size)
    a = rb(attn.reshape(T, q_w))
    h1 = rb(linear(a, w["w_o"]) + x.double().numpy())
    n2 = rb(rmsnorm(h1, w["g_mlp"], rms_eps))
    act = rb(swiglu_f64(linear(n2, w["w_gate"]), linear(n2, w["w_up"])))
    y = rb(linear(act, w["w_down"]) + h1.double().numpy())
    return dict(n=n, qkv=qkv, q=q, k=k, attn=a, h1=h1, n2=n2, act=act, y=y, k_cache=kc, v_cache=vc, cu_q=cu, pos=pos)


def model_verify(tok_id, embed, layers, g_final, w_lm, k_caches, v_caches, block_table, ctx_lens, depths, draft_ids,
                 n_q_heads, n_kv_heads, head_dim, page_size, rms_eps, rope_theta, return_stages=False):
    """The verification forward of a whole model on the retained tokens (Section 3.1: one packed target forward
    over each request's first d_i draft tokens, then acceptance): embedding lookup, `layer_forward` for every
    layer in turn (layer l with its own cache pair), final RMSNorm rounded to bf16, `lm_head_accept`.
    Returns (AcceptResult, logits fp64 [T, V], hidden: list of the bf16 hidden states after each layer, final
    normed states last, updated cache copies per layer); with `return_stages` also the list of `layer_forward`'s stage
    dicts, one per layer."""
    import torch
    tok_id = np.asarray(tok_id, np.int64)
    x = embed[torch.from_numpy(tok_id)]
    hidden, caches, stages = [], [], []
    cu = None
    for l, w in enumerate(layers):
        st = layer_forward(x, w, k_caches[l], v_caches[l], block_table, ctx_lens, depths, n_q_heads, n_kv_heads,
                           head_dim, page_size, rms_eps, rope_theta)
        x, cu = st["y"], st["cu_q"]
        hidden.append(x)
        caches.append((st["k_cache"], st["v_cache"]))
        stages.append(st)
    if cu is None:
        d = np.asarray(depths, np.int32)
        cu = np.zeros(len(d) + 1, np.int32)
        np.cumsum(d.astype(np.int64) + 1, out=cu[1:])
    n = _as_bf16_tensor(round_bf16(rmsnorm(x, g_final, rms_eps)))
    hidden.append(n)
    gamma = np.asarray(draft_ids).shape[1]
    res, logits64 = lm_head_accept(n, w_lm, draft_ids, cu, gamma)
    if return_stages:
        return res, logits64, hidden, caches, stages
    return res, logits64, hidden, caches
