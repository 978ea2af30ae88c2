"""Seeded synthetic inputs for the D-cut verify hot path.

This module only *draws inputs*.  It holds none of the method's arithmetic (no prefix
scores, no ranking, no attention, no argmax): the CPU oracle and the CUDA path both
consume what is generated here and each computes the method on its own.

The five workloads are stand-ins for the paper's high-concurrency serving setups
(Section 4.1: Qwen3-8B-class and Hy3-class GQA shapes, concurrency up to 64 and beyond,
block of 16 draft positions).  The paper's datasets, prompts and weights are not used.
Structure taken from the paper: acceptance decays along the block and varies strongly
across requests (Section 2.1), and drafter confidence tracks acceptance (Appendix E),
hence Beta-distributed confidences with a geometric decay and a planted reject index
whose distribution is tied to each request's mean confidence.

All draws use numpy's PCG64 (`numpy.random.default_rng`) with documented keys:

  default_rng([seed, TAG])            one stream per input family
  default_rng([seed, TAG, i, t])      one stream per (request i, block position t) row

so that a row for (i, t) is the same whatever depth vector packs it.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional, Tuple

import numpy as np
import torch

# stream tags
_TAG_CONF, _TAG_IDS, _TAG_CTX, _TAG_REJECT, _TAG_PAGES, _TAG_KV, _TAG_Q, _TAG_LOGITS = range(1, 9)
_TAG_LAYER_X, _TAG_LAYER_W = 9, 10
_TAG_LM_W, _TAG_LM_X = 11, 12
_TAG_DRAFT_LOGITS, _TAG_UNIFORM = 13, 14
_TAG_EMBED, _TAG_G_FINAL = 15, 16


@dataclass(frozen=True)
class WorkloadConfig:
    index: int
    name: str
    B: int
    gamma: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    page_size: int
    vocab: int
    conf_kind: str            # "beta_decay" | "skew_halves"
    conf_a: float = 0.0
    conf_b: float = 0.0
    conf_decay: float = 1.0
    ctx_kind: str = "uniform"  # "uniform" | "lognormal"
    ctx_lo: int = 0
    ctx_hi: int = 0
    ctx_median: float = 0.0
    ctx_sigma: float = 0.0
    hidden: int = 0            # layer configuration only
    intermediate: int = 0
    rope_theta: float = 1.0e6
    rms_eps: float = 1.0e-6

    @property
    def seed(self) -> int:
        return self.index

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def t_cap(self) -> int:
        return self.B * (self.gamma + 1)


CONFIGS: Tuple[WorkloadConfig, ...] = (
    WorkloadConfig(0, "tiny_b4", 4, 16, 4, 1, 64, 16, 32000, "beta_decay", 8.0, 2.0, 0.97,
                   "uniform", 64, 256),
    WorkloadConfig(1, "b16_ctx1k4k", 16, 16, 32, 8, 128, 16, 151936, "beta_decay", 6.0, 2.0, 0.95,
                   "uniform", 1024, 4096),
    WorkloadConfig(2, "b64_ctx2k8k_skew", 64, 16, 32, 8, 128, 16, 151936, "skew_halves", 0.0, 0.0, 1.0,
                   "uniform", 2048, 8192),
    WorkloadConfig(3, "b256_lognormal", 256, 16, 64, 8, 128, 16, 151936, "beta_decay", 5.0, 2.0, 0.95,
                   "lognormal", 512, 32768, 4096.0, 1.0),
    WorkloadConfig(4, "layer_b64", 64, 16, 32, 8, 128, 16, 151936, "skew_halves", 0.0, 0.0, 1.0,
                   "uniform", 2048, 8192, hidden=4096, intermediate=12288),
)


def config(index: int) -> WorkloadConfig:
    return CONFIGS[index]


def custom_config(**kw) -> WorkloadConfig:
    """A config for tests (edge shapes); unspecified fields follow the tiny config."""
    base = dict(index=100, name="custom", B=4, gamma=16, n_q_heads=4, n_kv_heads=1, head_dim=64,
                page_size=16, vocab=32000, conf_kind="beta_decay", conf_a=8.0, conf_b=2.0,
                conf_decay=0.97, ctx_kind="uniform", ctx_lo=64, ctx_hi=256)
    base.update(kw)
    return WorkloadConfig(**base)


# --------------------------------------------------------------------------- selection inputs

@dataclass
class SelectInputs:
    conf: np.ndarray        # fp32 [B, gamma]   drafter confidence c_{i,j}, j = 1..gamma
    draft_ids: np.ndarray   # i32  [B, gamma]   z_{i,1..gamma}
    bonus_ids: np.ndarray   # i32  [B]          z_{i,0}
    ctx_lens: np.ndarray    # i32  [B]          L_i: tokens already cached (bonus and drafts excluded)
    reject_index: np.ndarray  # i32 [B]         planted number of drafts the target would accept


def select_inputs(cfg: WorkloadConfig) -> SelectInputs:
    B, g = cfg.B, cfg.gamma
    rng = np.random.default_rng([cfg.seed, _TAG_CONF])
    if cfg.conf_kind == "beta_decay":
        raw = rng.beta(cfg.conf_a, cfg.conf_b, size=(B, g))
    elif cfg.conf_kind == "skew_halves":
        hi = rng.beta(9.0, 1.0, size=(B, g))
        lo = rng.beta(2.0, 3.0, size=(B, g))
        is_hi = (np.arange(B) % 2 == 0)[:, None]   # interleaved halves: even requests confident
        raw = np.where(is_hi, hi, lo)
    else:
        raise ValueError(cfg.conf_kind)
    j = np.arange(1, g + 1, dtype=np.float64)
    conf64 = raw * np.power(cfg.conf_decay, j)[None, :]
    conf = conf64.astype(np.float32)

    rng = np.random.default_rng([cfg.seed, _TAG_IDS])
    draft_ids = rng.integers(0, cfg.vocab, size=(B, g), dtype=np.int64).astype(np.int32)
    bonus_ids = rng.integers(0, cfg.vocab, size=(B,), dtype=np.int64).astype(np.int32)

    rng = np.random.default_rng([cfg.seed, _TAG_CTX])
    if cfg.ctx_kind == "uniform":
        ctx = rng.integers(cfg.ctx_lo, cfg.ctx_hi + 1, size=(B,), dtype=np.int64)
    elif cfg.ctx_kind == "lognormal":
        ctx = np.exp(rng.normal(np.log(cfg.ctx_median), cfg.ctx_sigma, size=(B,)))
        ctx = np.clip(np.rint(ctx), cfg.ctx_lo, cfg.ctx_hi).astype(np.int64)
    else:
        raise ValueError(cfg.ctx_kind)
    ctx_lens = ctx.astype(np.int32)

    # planted reject index: number of accepted drafts ~ Geometric(p) - 1, p = 1 - mean_j c_{i,j}
    rng = np.random.default_rng([cfg.seed, _TAG_REJECT])
    p = np.maximum(1.0e-3, 1.0 - conf.astype(np.float64).mean(axis=1))
    reject = np.minimum(rng.geometric(p) - 1, g).astype(np.int32)
    return SelectInputs(conf, draft_ids, bonus_ids, ctx_lens, reject)


def cost_table_linear(n: int, base_ms: float, slope_ms: float, knee: int = 0) -> np.ndarray:
    """cost_ms[T] = base + slope * max(0, T - knee), T = 0..n-1, as fp32."""
    T = np.arange(n, dtype=np.float64)
    return (base_ms + slope_ms * np.maximum(0.0, T - knee)).astype(np.float32)


def cost_table_for(cfg: WorkloadConfig) -> np.ndarray:
    """The analytic table of the tiny config; a linear stand-in elsewhere (the bench
    replaces it with the table profiled on the GPU)."""
    n = cfg.t_cap + 1
    if cfg.index == 0:
        return cost_table_linear(n, 10.0, 0.02, 64)
    return cost_table_linear(n, 0.2, 0.0003, 0)


# --------------------------------------------------------------------------- paged KV cache

@dataclass
class PagedKV:
    k_cache: torch.Tensor      # bf16 [num_pages, n_kv_heads, page_size, head_dim]
    v_cache: torch.Tensor      # bf16 same shape
    block_table: np.ndarray    # i32 [B, max_pages_per_req], unused slots = -1
    num_pages: int
    max_pages_per_req: int


def _randn_bf16(rng: np.random.Generator, n: int, chunk: int = 1 << 24) -> torch.Tensor:
    out = torch.empty(n, dtype=torch.bfloat16)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        out[s:e] = torch.from_numpy(rng.standard_normal(e - s, dtype=np.float32)).to(torch.bfloat16)
    return out


def paged_kv(cfg: WorkloadConfig, ctx_lens: np.ndarray, extra_pages: int = 3, layer: int = 0) -> PagedKV:
    """KV cache holding, per request, L_i cached tokens plus the gamma+1 block positions
    (bonus and all drafts: the caller appends them before verification, whatever depth
    is later kept).  Physical pages are assigned by a seeded permutation; the last page
    of a request is partially filled and its unused slots hold ordinary random values.
    `layer` > 0 gives another layer's cache: same block table, different contents."""
    B, ps = len(ctx_lens), cfg.page_size
    n_tok = ctx_lens.astype(np.int64) + cfg.gamma + 1
    n_pg = (n_tok + ps - 1) // ps
    total = int(n_pg.sum()) + extra_pages
    max_pages = int(n_pg.max())
    rng = np.random.default_rng([cfg.seed, _TAG_PAGES])
    perm = rng.permutation(total).astype(np.int32)
    bt = np.full((B, max_pages), -1, dtype=np.int32)
    o = 0
    for i in range(B):
        bt[i, : n_pg[i]] = perm[o : o + n_pg[i]]
        o += int(n_pg[i])
    rng = np.random.default_rng([cfg.seed, _TAG_KV] + ([layer] if layer else []))
    shape = (total, cfg.n_kv_heads, ps, cfg.head_dim)
    n = int(np.prod(shape))
    k = _randn_bf16(rng, n).view(shape)
    v = _randn_bf16(rng, n).view(shape)
    return PagedKV(k, v, bt, total, max_pages)


# --------------------------------------------------------------------------- packed rows

def cu_q_from_depths(depths: np.ndarray) -> np.ndarray:
    cu = np.zeros(len(depths) + 1, dtype=np.int32)
    np.cumsum(np.asarray(depths, dtype=np.int64) + 1, out=cu[1:])
    return cu


def q_rows(cfg: WorkloadConfig, depths: np.ndarray) -> torch.Tensor:
    """Query rows bf16 [T, n_q_heads, head_dim] ~ N(0,1), packed request-major; the row
    of (i, t) does not depend on the depth vector."""
    cu = cu_q_from_depths(depths)
    T = int(cu[-1])
    out = torch.empty((T, cfg.n_q_heads, cfg.head_dim), dtype=torch.bfloat16)
    for i, d in enumerate(depths):
        for t in range(int(d) + 1):
            rng = np.random.default_rng([cfg.seed, _TAG_Q, i, t])
            r = rng.standard_normal(cfg.n_q_heads * cfg.head_dim, dtype=np.float32)
            out[cu[i] + t] = torch.from_numpy(r).to(torch.bfloat16).view(cfg.n_q_heads, cfg.head_dim)
    return out


def logits_rows(cfg: WorkloadConfig, sel: SelectInputs, depths: np.ndarray,
                vocab: Optional[int] = None) -> torch.Tensor:
    """Target logits bf16 [T, V] ~ N(0,1), packed like `q_rows`.  On rows t < reject_index[i]
    the logit of the next draft token z_{i,t+1} is set to 8.0 (exact in bf16), which makes
    it the unique maximum: the target 'accepts' exactly reject_index[i] drafts."""
    V = cfg.vocab if vocab is None else vocab
    cu = cu_q_from_depths(depths)
    T = int(cu[-1])
    out = torch.empty((T, V), dtype=torch.bfloat16)
    for i, d in enumerate(depths):
        for t in range(int(d) + 1):
            rng = np.random.default_rng([cfg.seed, _TAG_LOGITS, i, t])
            r = torch.from_numpy(rng.standard_normal(V, dtype=np.float32)).to(torch.bfloat16)
            if t < int(sel.reject_index[i]) and t < cfg.gamma:
                r[int(sel.draft_ids[i, t]) % V] = 8.0
            out[cu[i] + t] = r
    return out


# --------------------------------------------------------------------------- decoder layer inputs

@dataclass
class LayerWeights:
    w_qkv: torch.Tensor    # bf16 [(Hq + 2 Hkv) * Dh, hidden]   rows: q heads, then k heads, then v heads
    w_o: torch.Tensor      # bf16 [hidden, Hq * Dh]
    w_gate: torch.Tensor   # bf16 [intermediate, hidden]
    w_up: torch.Tensor     # bf16 [intermediate, hidden]
    w_down: torch.Tensor   # bf16 [hidden, intermediate]
    g_attn: torch.Tensor   # bf16 [hidden]  RMSNorm gain before attention
    g_mlp: torch.Tensor    # bf16 [hidden]  RMSNorm gain before the MLP


def layer_weights(cfg: WorkloadConfig, hidden: Optional[int] = None,
                  intermediate: Optional[int] = None, layer: int = 0) -> LayerWeights:
    """Random-init weights ~ N(0, 0.02^2), gains ~ 1 + N(0, 0.02^2), bf16; `layer` > 0 draws another layer's set."""
    H = cfg.hidden if hidden is None else hidden
    I = cfg.intermediate if intermediate is None else intermediate
    rng = np.random.default_rng([cfg.seed, _TAG_LAYER_W] + ([layer] if layer else []))

    def w(r, c):
        return (_randn_bf16(rng, r * c).float() * 0.02).to(torch.bfloat16).view(r, c)

    qkv_rows = (cfg.n_q_heads + 2 * cfg.n_kv_heads) * cfg.head_dim
    w_qkv = w(qkv_rows, H)
    w_o = w(H, cfg.n_q_heads * cfg.head_dim)
    w_gate = w(I, H)
    w_up = w(I, H)
    w_down = w(H, I)
    g1 = (1.0 + 0.02 * _randn_bf16(rng, H).float()).to(torch.bfloat16)
    g2 = (1.0 + 0.02 * _randn_bf16(rng, H).float()).to(torch.bfloat16)
    return LayerWeights(w_qkv, w_o, w_gate, w_up, w_down, g1, g2)


def layer_x_rows(cfg: WorkloadConfig, depths: np.ndarray, hidden: Optional[int] = None) -> torch.Tensor:
    """Layer input bf16 [T, hidden] ~ N(0,1), one counter-seeded row per (i, t)."""
    H = cfg.hidden if hidden is None else hidden
    cu = cu_q_from_depths(depths)
    out = torch.empty((int(cu[-1]), H), dtype=torch.bfloat16)
    for i, d in enumerate(depths):
        for t in range(int(d) + 1):
            rng = np.random.default_rng([cfg.seed, _TAG_LAYER_X, i, t])
            out[cu[i] + t] = torch.from_numpy(rng.standard_normal(H, dtype=np.float32)).to(torch.bfloat16)
    return out


# --------------------------------------------------------------------------- LM head inputs

def lm_head_weight(cfg: WorkloadConfig, vocab: Optional[int] = None, hidden: Optional[int] = None) -> torch.Tensor:
    """LM-head weight bf16 [V, hidden] ~ N(0, 0.02^2)."""
    V = cfg.vocab if vocab is None else vocab
    H = cfg.hidden if hidden is None else hidden
    rng = np.random.default_rng([cfg.seed, _TAG_LM_W])
    return (_randn_bf16(rng, V * H).float().mul_(0.02)).to(torch.bfloat16).view(V, H)


def lm_head_x_rows(cfg: WorkloadConfig, sel: SelectInputs, depths: np.ndarray, w_lm: torch.Tensor) -> torch.Tensor:
    """Last hidden states bf16 [T, hidden], packed like `q_rows`.  Rows t < reject_index[i] are 5 x the LM-head row of
    the next draft token z_{i,t+1}, which makes that token the maximum by a wide margin (the target 'accepts' exactly
    reject_index[i] drafts); every other row is ~ N(0,1), one counter-seeded draw per (i, t)."""
    V, H = w_lm.shape
    cu = cu_q_from_depths(depths)
    out = torch.empty((int(cu[-1]), H), dtype=torch.bfloat16)
    for i, d in enumerate(depths):
        for t in range(int(d) + 1):
            if t < int(sel.reject_index[i]) and t < cfg.gamma:
                out[cu[i] + t] = (w_lm[int(sel.draft_ids[i, t]) % V].float() * 5.0).to(torch.bfloat16)
            else:
                rng = np.random.default_rng([cfg.seed, _TAG_LM_X, i, t])
                out[cu[i] + t] = torch.from_numpy(rng.standard_normal(H, dtype=np.float32)).to(torch.bfloat16)
    return out


# --------------------------------------------------------------------------- whole-model inputs

@dataclass
class ModelWeights:
    embed: torch.Tensor        # bf16 [V, hidden] ~ N(0, 1): the hidden states enter the first layer at unit scale
    layers: list               # LayerWeights per layer
    g_final: torch.Tensor      # bf16 [hidden]
    w_lm: torch.Tensor         # bf16 [V, hidden]


def model_weights(cfg: WorkloadConfig, n_layers: int, vocab: Optional[int] = None, hidden: Optional[int] = None,
                  intermediate: Optional[int] = None) -> ModelWeights:
    """Random-init weights of a small decoder-only model (untied embedding and LM head)."""
    V = cfg.vocab if vocab is None else vocab
    H = cfg.hidden if hidden is None else hidden
    embed = _randn_bf16(np.random.default_rng([cfg.seed, _TAG_EMBED]), V * H).view(V, H)
    g = (1.0 + 0.02 * _randn_bf16(np.random.default_rng([cfg.seed, _TAG_G_FINAL]), H).float()).to(torch.bfloat16)
    return ModelWeights(embed, [layer_weights(cfg, H, intermediate, layer=l) for l in range(n_layers)], g,
                        lm_head_weight(cfg, V, H))


def model_tok_ids(sel: SelectInputs, depths: np.ndarray, vocab: int) -> np.ndarray:
    """The packed input tokens of the verification forward: per request the previous step's bonus token, then its
    first d_i draft tokens (ids folded into [0, vocab))."""
    return np.concatenate([np.concatenate([[sel.bonus_ids[i]], sel.draft_ids[i, : int(d)]])
                           for i, d in enumerate(depths)]).astype(np.int64) % vocab


# --------------------------------------------------------------------------- stochastic variant inputs

def draft_logits_rows(cfg: WorkloadConfig, target_rows: torch.Tensor, depths: np.ndarray, noise: float = 0.7,
                      vocab: Optional[int] = None) -> torch.Tensor:
    """Drafter logits bf16 [B, gamma, V]: row (i, t) = the target row that verifies draft t + 1 of request i plus
    N(0, noise^2) per token (a drafter that tracks the target imperfectly, so p(z)/q(z) scatters around 1); rows
    t >= d_i have no target row and are ~ N(0, 1).  One counter-seeded draw per (i, t)."""
    V = cfg.vocab if vocab is None else vocab
    cu = cu_q_from_depths(depths)
    out = torch.empty((cfg.B, cfg.gamma, V), dtype=torch.bfloat16)
    for i, d in enumerate(depths):
        for t in range(cfg.gamma):
            rng = np.random.default_rng([cfg.seed, _TAG_DRAFT_LOGITS, i, t])
            r = torch.from_numpy(rng.standard_normal(V, dtype=np.float32))
            if t < int(d):
                r = target_rows[cu[i] + t].float() + noise * r
            out[i, t] = r.to(torch.bfloat16)
    return out


def uniforms(cfg: WorkloadConfig):
    """The random numbers of rejection-sampling acceptance: u_accept fp32 [B, gamma], u_sample fp32 [B], in [0, 1)."""
    rng = np.random.default_rng([cfg.seed, _TAG_UNIFORM])
    return rng.random((cfg.B, cfg.gamma), dtype=np.float32), rng.random(cfg.B, dtype=np.float32)
