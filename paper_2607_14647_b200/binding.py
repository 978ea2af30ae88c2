"""Thin ctypes binding of libdcut.so: argument marshalling only.

Each function has the name and meaning of the C entry point declared in include/dcut.h; tensors
are torch CUDA tensors whose `data_ptr()` is passed through, the stream is torch's current
stream.  There is no CPU fallback: importing this module without a built library raises, and
every call runs the CUDA kernels.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdcut.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is not built; run `python -m paper_2607_14647_b200.build` "
                      "(needs nvcc; there is no fallback path)")
_lib = C.CDLL(LIB_PATH)

OK, EINVAL, ECAPACITY, ECUDA, ECOST, EDEVICE = range(6)
STATUS_NAMES = ["DCUT_OK", "DCUT_EINVAL", "DCUT_ECAPACITY", "DCUT_ECUDA", "DCUT_ECOST", "DCUT_EDEVICE"]

EXPORTS = ["dcut_create", "dcut_destroy", "dcut_last_error", "dcut_set_cost_dense", "dcut_set_cost_buckets",
           "dcut_budget_from_ratio", "dcut_select", "dcut_verify_attn", "dcut_accept", "dcut_verify_step_host",
           "dcut_accept_static", "dcut_gemm_bf16", "dcut_layer_forward", "dcut_lm_head_accept",
           "dcut_select_causal", "dcut_accept_rs", "dcut_commit", "dcut_model_verify", "dcut_poll_device_status",
           "dcut_enable_plan_in_select", "dcut_cost_grid_create", "dcut_cost_grid_destroy", "dcut_cost_grid_budget",
           "dcut_cost_grid_record", "dcut_cost_grid_get", "dcut_cost_grid_nearest", "dcut_cost_grid_buckets",
           "dcut_set_cost_from_grid", "dcut_layer_attn_part", "dcut_layer_mlp_part", "dcut_residual_add"]


class Limits(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("max_B", "max_gamma", "n_q_heads", "n_kv_heads", "head_dim", "page_size",
                                       "max_pages_per_req", "vocab", "hidden", "intermediate")]


class SelectInfo(C.Structure):
    _fields_ = [("n_star", C.c_int32), ("t_total", C.c_int32), ("candidate", C.c_int32), ("reserved", C.c_int32),
                ("sum_fixed", C.c_int64), ("objective", C.c_double)]


_vp, _i, _ll, _f = C.c_void_p, C.c_int, C.c_longlong, C.c_float


class HostStep(C.Structure):
    _fields_ = [("B", _i), ("gamma", _i), ("vocab", _i), ("block_table_stride", _i), ("num_pages", _ll),
                ("scale", _f)] + [(n, _vp) for n in (
                    "conf", "draft_ids", "bonus_ids", "ctx_lens", "block_table", "q_rows", "logits_rows", "k_cache",
                    "v_cache", "depths", "accept_len", "bonus", "out_tokens", "n_accepted_total", "attn_out",
                    "h2d_bytes", "d2h_bytes", "hidden_rows", "w_lm")]


_lib.dcut_verify_step_host.argtypes = [_vp, C.POINTER(HostStep), _vp]
_lib.dcut_create.argtypes = [C.POINTER(_vp), C.POINTER(Limits), _i]
_lib.dcut_destroy.argtypes = [_vp]
_lib.dcut_last_error.argtypes = [_vp]
_lib.dcut_last_error.restype = C.c_char_p
_lib.dcut_set_cost_dense.argtypes = [_vp, _vp, _i]
_lib.dcut_set_cost_buckets.argtypes = [_vp, _i, _i, _vp, _vp, _i]
_lib.dcut_budget_from_ratio.argtypes = [_i, _i, _i, _i, C.POINTER(_i)]
_lib.dcut_select.argtypes = [_vp, _vp, _i, _i] + [_vp] * 11 + [_vp]
_lib.dcut_select_causal.argtypes = [_vp, _vp, _i, _i] + [_vp] * 11 + [_vp]
_lib.dcut_enable_plan_in_select.argtypes = [_vp, _i]
_lib.dcut_cost_grid_create.argtypes = [C.POINTER(_vp), _vp, _i, _vp, _vp, _i, _i]
_lib.dcut_cost_grid_destroy.argtypes = [_vp]
_lib.dcut_cost_grid_budget.argtypes = [_vp, _i, _i, C.POINTER(_i)]
_lib.dcut_cost_grid_record.argtypes = [_vp, _i, _i, _vp, _i]
_lib.dcut_cost_grid_get.argtypes = [_vp, _i, _i, C.POINTER(_f)]
_lib.dcut_cost_grid_nearest.argtypes = [_vp, _i, C.POINTER(_i)]
_lib.dcut_cost_grid_buckets.argtypes = [_vp, _i, _vp, _vp, C.POINTER(_i)]
_lib.dcut_set_cost_from_grid.argtypes = [_vp, _vp, _i]
_lib.dcut_accept_rs.argtypes = [_vp, _vp, _vp, _i, _vp, _vp, _i, _i, _i] + [_vp] * 8
_lib.dcut_commit.argtypes = [_vp, _vp, _vp, _i, _i, _i, _vp, _vp, _vp, _vp, _i, _vp]
_lib.dcut_verify_attn.argtypes = [_vp, _vp, _vp, _vp, _ll, _vp, _i, _vp, _vp, _i, _i, _f, _vp, _vp, _vp]
_lib.dcut_accept.argtypes = [_vp, _vp, _i, _vp, _vp, _i, _i, _i, _vp, _vp, _vp, _vp, _vp]
_lib.dcut_poll_device_status.argtypes = [_vp, C.POINTER(_i), _vp]


_lib.dcut_accept_static.argtypes = [_vp, _i, _vp, _vp, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, C.c_char_p, C.c_size_t]
ACCEPT_STATIC_MAX_ROWS = 8192


class LayerWeights(C.Structure):
    _fields_ = [(n, _vp) for n in ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")] + \
               [("rms_eps", _f), ("rope_theta", _f)]


class Model(C.Structure):
    _fields_ = [("n_layers", _i), ("layers", C.POINTER(LayerWeights)), ("k_caches", C.POINTER(_vp)),
                ("v_caches", C.POINTER(_vp)), ("embed", _vp), ("g_final", _vp), ("w_lm", _vp), ("vocab", _i)]


_lib.dcut_model_verify.argtypes = [_vp, C.POINTER(Model), _ll, _vp, _i, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i,
                                   _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.dcut_gemm_bf16.argtypes = [_vp, _vp, _vp, _vp, _i, _i, _i, _vp, _i, _i, _vp, _vp, _vp]
_lib.dcut_lm_head_accept.argtypes = [_vp, _vp, _vp, _i, _vp, _vp, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.dcut_layer_forward.argtypes = [_vp, C.POINTER(LayerWeights), _vp, _vp, _vp, _vp, _ll, _vp, _i, _vp, _vp, _vp, _vp,
                                    _i, _i, _vp]
_lib.dcut_layer_attn_part.argtypes = _lib.dcut_layer_forward.argtypes
_lib.dcut_layer_mlp_part.argtypes = [_vp, C.POINTER(LayerWeights), _vp, _vp, _vp, _i, _i, _vp]
_lib.dcut_residual_add.argtypes = [_vp, _vp, _vp, _vp, _i, _vp, _i, _i, _vp]


@dataclass
class PreparedModel:
    rec: "Model"
    keep: tuple              # the ctypes arrays and tensors `rec` points into
    num_pages: int
    device: torch.device


class DcutError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"{STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else status}: {msg}")
        self.status = status


def _ptr(t: Optional[torch.Tensor], dtype=None) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    if dtype is not None:
        assert t.dtype == dtype, f"expected {dtype}, got {t.dtype}"
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def budget_from_ratio(B: int, gamma: int, num: int, den: int) -> int:
    k = _i(0)
    st = _lib.dcut_budget_from_ratio(B, gamma, num, den, C.byref(k))
    if st != OK:
        raise DcutError(st, "dcut_budget_from_ratio")
    return k.value


def accept_static(logits, draft_ids, cu_q, T_cap: int, accept_len, bonus, out_tokens, total):
    """dcut_accept_static: acceptance for callers that may not allocate (no context, fixed scratch inside the
    library, at most ACCEPT_STATIC_MAX_ROWS packed rows).  All tensors are the caller's CUDA tensors."""
    B, gamma = draft_ids.shape
    err = C.create_string_buffer(256)
    st = _lib.dcut_accept_static(_ptr(logits, torch.bfloat16), logits.shape[1], _ptr(draft_ids, torch.int32),
                                 _ptr(cu_q, torch.int32), B, gamma, T_cap, _ptr(accept_len), _ptr(bonus),
                                 _ptr(out_tokens), _ptr(total), _stream(), err, len(err))
    if st != OK:
        raise DcutError(st, err.value.decode())


@dataclass
class SelectOut:
    depths: torch.Tensor
    cu_q: torch.Tensor
    tok_req: torch.Tensor
    tok_pos: torch.Tensor
    tok_id: torch.Tensor
    info: torch.Tensor       # int64 [4] view of dcut_select_info: see `read_info`
    scores: Optional[torch.Tensor]
    ranks: Optional[torch.Tensor]


class CostGrid:
    """dcut_cost_grid: the start-up cost table C(B, rho), a host object (works without a GPU)."""

    def __init__(self, batch_sizes: Sequence[int], ratios: Sequence[Tuple[int, int]], gamma: int):
        self.batch_sizes, self.ratios, self.gamma = [int(b) for b in batch_sizes], [(int(n), int(d)) for n, d in ratios], int(gamma)
        b = np.ascontiguousarray(self.batch_sizes, dtype=np.int32)
        num = np.ascontiguousarray([r[0] for r in self.ratios], dtype=np.int32)
        den = np.ascontiguousarray([r[1] for r in self.ratios], dtype=np.int32)
        self._h = _vp(None)
        st = _lib.dcut_cost_grid_create(C.byref(self._h), b.ctypes.data, len(b), num.ctypes.data, den.ctypes.data, len(num), gamma)
        if st != OK:
            raise DcutError(st, "dcut_cost_grid_create: batch sizes and ratios must ascend; ratios in (0, 1]; gamma >= 1")

    def close(self):
        if getattr(self, "_h", None):
            _lib.dcut_cost_grid_destroy(self._h)
            self._h = _vp(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int, what: str):
        if st != OK:
            raise DcutError(st, what)

    def budget(self, B: int, r: int) -> int:
        k = _i(0)
        self._check(_lib.dcut_cost_grid_budget(self._h, B, r, C.byref(k)), "dcut_cost_grid_budget")
        return k.value

    def record(self, b: int, r: int, samples_ms: Sequence[float]):
        a = np.ascontiguousarray(samples_ms, dtype=np.float32)
        self._check(_lib.dcut_cost_grid_record(self._h, b, r, a.ctypes.data, len(a)), "dcut_cost_grid_record: bad cell or sample")

    def get(self, b: int, r: int) -> float:
        v = _f(0.0)
        self._check(_lib.dcut_cost_grid_get(self._h, b, r, C.byref(v)), "dcut_cost_grid_get")
        return v.value

    def table(self) -> np.ndarray:
        return np.array([[self.get(b, r) for r in range(len(self.ratios))] for b in range(len(self.batch_sizes))], np.float32)

    def nearest(self, B: int) -> int:
        b = _i(0)
        self._check(_lib.dcut_cost_grid_nearest(self._h, B, C.byref(b)), "dcut_cost_grid_nearest")
        return b.value

    def buckets(self, B: int):
        K = np.zeros(len(self.ratios), np.int32)
        c = np.zeros(len(self.ratios), np.float32)
        n = _i(0)
        self._check(_lib.dcut_cost_grid_buckets(self._h, B, K.ctypes.data, c.ctypes.data, C.byref(n)),
                    "dcut_cost_grid_buckets: the nearest row is not fully recorded")
        return K[: n.value].copy(), c[: n.value].copy()


def read_info(info: torch.Tensor) -> SelectInfo:
    """Copies the device record to the host (synchronises)."""
    raw = info.cpu().numpy().tobytes()
    return SelectInfo.from_buffer_copy(raw)


class Context:
    """Owns a dcut_ctx.  Calls are asynchronous on torch's current stream."""

    def __init__(self, max_B: int, max_gamma: int, n_q_heads: int = 0, n_kv_heads: int = 0, head_dim: int = 0,
                 page_size: int = 16, max_pages_per_req: int = 0, vocab: int = 0, hidden: int = 0,
                 intermediate: int = 0, device: Optional[int] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("libdcut needs a CUDA device (sm_100a); there is no CPU path")
        self.device = torch.cuda.current_device() if device is None else device
        self.limits = Limits(max_B, max_gamma, n_q_heads, n_kv_heads, head_dim, page_size, max_pages_per_req,
                             vocab, hidden, intermediate)
        self._h = _vp(None)
        st = _lib.dcut_create(C.byref(self._h), C.byref(self.limits), self.device)
        if st != OK:
            msg = _lib.dcut_last_error(self._h).decode() if self._h else "dcut_create"
            _lib.dcut_destroy(self._h)
            self._h = _vp(None)
            raise DcutError(st, msg)

    def close(self):
        if getattr(self, "_h", None):
            _lib.dcut_destroy(self._h)
            self._h = _vp(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int):
        if st != OK:
            raise DcutError(st, _lib.dcut_last_error(self._h).decode())

    # -- cost model (host arrays) ------------------------------------------------------------
    def set_cost_dense(self, cost_ms: Sequence[float]):
        a = np.ascontiguousarray(cost_ms, dtype=np.float32)
        self._check(_lib.dcut_set_cost_dense(self._h, a.ctypes.data, len(a)))

    def set_cost_buckets(self, B: int, gamma: int, K: Sequence[int], cost_ms: Sequence[float]):
        k = np.ascontiguousarray(K, dtype=np.int32)
        a = np.ascontiguousarray(cost_ms, dtype=np.float32)
        assert len(k) == len(a)
        self._check(_lib.dcut_set_cost_buckets(self._h, B, gamma, k.ctypes.data, a.ctypes.data, len(a)))

    def enable_plan_in_select(self, on: bool = True):
        """dcut_enable_plan_in_select: the selector also builds the attention work list of the batch it packs."""
        self._check(_lib.dcut_enable_plan_in_select(self._h, 1 if on else 0))

    def set_cost_from_grid(self, grid: "CostGrid", B: int):
        """dcut_set_cost_from_grid: bucket mode with the budgets of a live batch of B and the nearest captured row."""
        self._check(_lib.dcut_set_cost_from_grid(self._h, grid._h, B))

    # -- hot path ------------------------------------------------------------------------------
    def select(self, conf, draft_ids, bonus_ids, ctx_lens, out: Optional[SelectOut] = None,
               want_scores: bool = False, want_ranks: bool = False, causal: bool = False) -> SelectOut:
        """dcut_select, or dcut_select_causal (shifted scores + early-stopping scan) with causal=True."""
        B, gamma = conf.shape
        dev = conf.device
        if out is None:
            cap = B * (gamma + 1)
            i32 = dict(dtype=torch.int32, device=dev)
            out = SelectOut(torch.empty(B, **i32), torch.empty(B + 1, **i32), torch.empty(cap, **i32),
                            torch.empty(cap, **i32), torch.empty(cap, **i32),
                            torch.zeros(4, dtype=torch.int64, device=dev),
                            torch.empty((B, gamma), dtype=torch.float32, device=dev) if want_scores else None,
                            torch.empty((B, gamma), **i32) if want_ranks else None)
        fn = _lib.dcut_select_causal if causal else _lib.dcut_select
        self._check(fn(self._h, _ptr(conf, torch.float32), B, gamma, _ptr(draft_ids, torch.int32),
                                     _ptr(bonus_ids, torch.int32), _ptr(ctx_lens, torch.int32),
                                     _ptr(out.depths), _ptr(out.cu_q), _ptr(out.tok_req), _ptr(out.tok_pos),
                                     _ptr(out.tok_id), _ptr(out.info), _ptr(out.scores), _ptr(out.ranks), _stream()))
        return out

    def verify_attn(self, q, k_cache, v_cache, block_table, ctx_lens, cu_q, T_cap: int, scale: Optional[float] = None,
                    out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None) -> torch.Tensor:
        B = ctx_lens.shape[0]
        if out is None:
            out = torch.empty_like(q)
        if scale is None:
            scale = 1.0 / float(np.sqrt(self.limits.head_dim))
        self._check(_lib.dcut_verify_attn(self._h, _ptr(q, torch.bfloat16), _ptr(k_cache, torch.bfloat16),
                                          _ptr(v_cache, torch.bfloat16), k_cache.shape[0],
                                          _ptr(block_table, torch.int32), block_table.shape[1],
                                          _ptr(ctx_lens, torch.int32), _ptr(cu_q, torch.int32), B, T_cap,
                                          float(scale), _ptr(out, torch.bfloat16), _ptr(lse, torch.float32),
                                          _stream()))
        return out

    def commit(self, accept_len, out_tokens, ctx_lens, bonus_ids, max_ctx: int, stream_tokens=None, stream_len=None):
        """dcut_commit: advances ctx_lens in place, writes the next step's bonus_ids, appends to the token streams."""
        B, g1 = out_tokens.shape
        cap = stream_tokens.shape[1] if stream_tokens is not None else 0
        self._check(_lib.dcut_commit(self._h, _ptr(accept_len, torch.int32), _ptr(out_tokens, torch.int32), B, g1 - 1,
                                     max_ctx, _ptr(ctx_lens, torch.int32), _ptr(bonus_ids, torch.int32),
                                     _ptr(stream_tokens, torch.int32), _ptr(stream_len, torch.int32), cap, _stream()))

    def accept_rs(self, target_logits, draft_logits, draft_ids, cu_q, T_cap: int, u_accept, u_sample,
                  want_prob: bool = False):
        """dcut_accept_rs: rejection-sampling acceptance; returns (accept_len, sampled token, out_tokens, total, prob)."""
        B, gamma = draft_ids.shape
        V = target_logits.shape[1]
        dev_ = target_logits.device
        i32 = dict(dtype=torch.int32, device=dev_)
        accept_len, bonus = torch.empty(B, **i32), torch.empty(B, **i32)
        toks, total = torch.empty((B, gamma + 1), **i32), torch.empty(1, **i32)
        prob = torch.zeros((B, 2), dtype=torch.float32, device=dev_) if want_prob else None
        self._check(_lib.dcut_accept_rs(self._h, _ptr(target_logits, torch.bfloat16), _ptr(draft_logits, torch.bfloat16), V,
                                        _ptr(draft_ids, torch.int32), _ptr(cu_q, torch.int32), B, gamma, T_cap,
                                        _ptr(u_accept, torch.float32), _ptr(u_sample, torch.float32), _ptr(accept_len),
                                        _ptr(bonus), _ptr(toks), _ptr(total), _ptr(prob), _stream()))
        return accept_len, bonus, toks, total, prob

    def accept(self, logits, draft_ids, cu_q, T_cap: int, out_tokens: bool = True):
        B, gamma = draft_ids.shape
        V = logits.shape[1]
        i32 = dict(dtype=torch.int32, device=logits.device)
        accept_len, bonus = torch.empty(B, **i32), torch.empty(B, **i32)
        toks = torch.empty((B, gamma + 1), **i32) if out_tokens else None
        total = torch.empty(1, **i32)
        self.accept_into(logits, draft_ids, cu_q, T_cap, accept_len, bonus, toks, total)
        return accept_len, bonus, toks, total

    def accept_into(self, logits, draft_ids, cu_q, T_cap, accept_len, bonus, out_tokens, total):
        B, gamma = draft_ids.shape
        self._check(_lib.dcut_accept(self._h, _ptr(logits, torch.bfloat16), logits.shape[1],
                                     _ptr(draft_ids, torch.int32), _ptr(cu_q, torch.int32), B, gamma, T_cap,
                                     _ptr(accept_len), _ptr(bonus), _ptr(out_tokens), _ptr(total), _stream()))

    def verify_step_host(self, conf, draft_ids, bonus_ids, ctx_lens, block_table, q_rows, logits_rows, k_cache,
                         v_cache, out: Optional[dict] = None, scale: Optional[float] = None, want_attn_out=False,
                         hidden_rows=None, w_lm=None):
        """Whole step from HOST tensors (CPU torch tensors, ideally pinned); k_cache / v_cache are the
        device-resident cache.  Returns a dict of CPU tensors plus the bytes copied each way.
        Hidden-state form: logits_rows=None, hidden_rows (CPU bf16 [B, gamma+1, hidden]) and w_lm (CUDA bf16 [V, hidden])."""
        B, gamma = conf.shape
        V = logits_rows.shape[-1] if logits_rows is not None else w_lm.shape[0]
        for t in (conf, draft_ids, bonus_ids, ctx_lens, block_table, q_rows, logits_rows, hidden_rows):
            assert t is None or (not t.is_cuda and t.is_contiguous())
        if out is None:
            out = self.host_step_outputs(B, gamma, want_attn_out)
        if scale is None:
            scale = 1.0 / float(np.sqrt(self.limits.head_dim))
        h2d, d2h = _ll(0), _ll(0)
        hs = HostStep(B, gamma, V, block_table.shape[1], k_cache.shape[0], float(scale), conf.data_ptr(),
                      draft_ids.data_ptr(), bonus_ids.data_ptr(), ctx_lens.data_ptr(), block_table.data_ptr(),
                      q_rows.data_ptr(), logits_rows.data_ptr() if logits_rows is not None else None, _ptr(k_cache, torch.bfloat16),
                      _ptr(v_cache, torch.bfloat16), out["depths"].data_ptr(), out["accept_len"].data_ptr(),
                      out["bonus"].data_ptr(), out["out_tokens"].data_ptr(), out["n_accepted_total"].data_ptr(),
                      out["attn_out"].data_ptr() if out.get("attn_out") is not None else None,
                      C.addressof(h2d), C.addressof(d2h), hidden_rows.data_ptr() if hidden_rows is not None else None,
                      _ptr(w_lm, torch.bfloat16))
        self._check(_lib.dcut_verify_step_host(self._h, C.byref(hs), _stream()))
        out["h2d_bytes"], out["d2h_bytes"] = h2d.value, d2h.value
        return out

    def host_step_outputs(self, B: int, gamma: int, want_attn_out: bool = False) -> dict:
        pin = dict(dtype=torch.int32, pin_memory=True)
        out = dict(depths=torch.zeros(B, **pin), accept_len=torch.zeros(B, **pin), bonus=torch.zeros(B, **pin),
                   out_tokens=torch.zeros((B, gamma + 1), **pin), n_accepted_total=torch.zeros(1, **pin), attn_out=None)
        if want_attn_out:
            out["attn_out"] = torch.zeros((B * (gamma + 1), self.limits.n_q_heads, self.limits.head_dim),
                                          dtype=torch.bfloat16, pin_memory=True)
        return out

    def gemm_bf16(self, a, w, cu_q, T_cap: int, out, mode: int = 0, w2=None, residual=None):
        """out[T, N] = a[T, K] . w[N, K]^T; mode 1 adds `residual`; mode 2 is SwiGLU with gate w and up w2."""
        B = cu_q.shape[0] - 1
        N, K = w.shape
        self._check(_lib.dcut_gemm_bf16(self._h, _ptr(a, torch.bfloat16), _ptr(w, torch.bfloat16),
                                        _ptr(w2, torch.bfloat16), mode, N, K, _ptr(cu_q, torch.int32), B, T_cap,
                                        _ptr(out, torch.bfloat16), _ptr(residual, torch.bfloat16), _stream()))
        return out

    def lm_head_accept(self, x, w_lm, draft_ids, cu_q, T_cap: int, out_tokens: bool = True, row_argmax: bool = False):
        """dcut_lm_head_accept: acceptance straight from the last hidden states x[T, hidden] and the LM head w_lm[V, hidden]."""
        B, gamma = draft_ids.shape
        V = w_lm.shape[0]
        i32 = dict(dtype=torch.int32, device=x.device)
        accept_len, bonus = torch.empty(B, **i32), torch.empty(B, **i32)
        toks = torch.empty((B, gamma + 1), **i32) if out_tokens else None
        total = torch.empty(1, **i32)
        am = torch.full((T_cap,), -1, **i32) if row_argmax else None
        self._check(_lib.dcut_lm_head_accept(self._h, _ptr(x, torch.bfloat16), _ptr(w_lm, torch.bfloat16), V,
                                             _ptr(draft_ids, torch.int32), _ptr(cu_q, torch.int32), B, gamma, T_cap,
                                             _ptr(accept_len), _ptr(bonus), _ptr(toks), _ptr(total), _ptr(am), _stream()))
        return accept_len, bonus, toks, total, am

    def layer_forward(self, weights: dict, x, y, k_cache, v_cache, block_table, ctx_lens, cu_q, tok_req, tok_pos,
                      T_cap: int, rms_eps: float = 1e-6, rope_theta: float = 1e6):
        """dcut_layer_forward; `weights` maps w_qkv, w_o, w_gate, w_up, w_down, g_attn, g_mlp to CUDA bf16 tensors."""
        lw = LayerWeights(*[_ptr(weights[n], torch.bfloat16) for n in
                            ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")], rms_eps, rope_theta)
        B = ctx_lens.shape[0]
        self._check(_lib.dcut_layer_forward(self._h, C.byref(lw), _ptr(x, torch.bfloat16), _ptr(y, torch.bfloat16),
                                            _ptr(k_cache, torch.bfloat16), _ptr(v_cache, torch.bfloat16),
                                            k_cache.shape[0], _ptr(block_table, torch.int32), block_table.shape[1],
                                            _ptr(ctx_lens, torch.int32), _ptr(cu_q, torch.int32),
                                            _ptr(tok_req, torch.int32), _ptr(tok_pos, torch.int32), B, T_cap, _stream()))
        return y

    def layer_attn_part(self, weights: dict, x, o_part, k_cache, v_cache, block_table, ctx_lens, cu_q, tok_req, tok_pos,
                        T_cap: int, rms_eps: float = 1e-6, rope_theta: float = 1e6):
        """dcut_layer_attn_part: a tensor-parallel rank's attention half of the layer (its partial O projection, no residual)."""
        lw = LayerWeights(*[_ptr(weights[n], torch.bfloat16) for n in
                            ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")], rms_eps, rope_theta)
        B = ctx_lens.shape[0]
        self._check(_lib.dcut_layer_attn_part(self._h, C.byref(lw), _ptr(x, torch.bfloat16), _ptr(o_part, torch.bfloat16),
                                              _ptr(k_cache, torch.bfloat16), _ptr(v_cache, torch.bfloat16),
                                              k_cache.shape[0], _ptr(block_table, torch.int32), block_table.shape[1],
                                              _ptr(ctx_lens, torch.int32), _ptr(cu_q, torch.int32),
                                              _ptr(tok_req, torch.int32), _ptr(tok_pos, torch.int32), B, T_cap, _stream()))
        return o_part

    def layer_mlp_part(self, weights: dict, h1, d_part, cu_q, T_cap: int, rms_eps: float = 1e-6, rope_theta: float = 1e6):
        """dcut_layer_mlp_part: the rank's MLP half (its partial down projection, no residual)."""
        lw = LayerWeights(*[_ptr(weights[n], torch.bfloat16) for n in
                            ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")], rms_eps, rope_theta)
        self._check(_lib.dcut_layer_mlp_part(self._h, C.byref(lw), _ptr(h1, torch.bfloat16), _ptr(d_part, torch.bfloat16),
                                             _ptr(cu_q, torch.int32), cu_q.shape[0] - 1, T_cap, _stream()))
        return d_part

    def residual_add(self, a, b, out, cu_q, T_cap: int):
        """dcut_residual_add: out = a + b over the packed rows in use."""
        self._check(_lib.dcut_residual_add(self._h, _ptr(a, torch.bfloat16), _ptr(b, torch.bfloat16), _ptr(out, torch.bfloat16),
                                           a.shape[1], _ptr(cu_q, torch.int32), cu_q.shape[0] - 1, T_cap, _stream()))
        return out

    def make_model(self, layers: list, embed, g_final, w_lm, k_caches: list, v_caches: list, rms_eps: float = 1e-6,
                   rope_theta: float = 1e6) -> "PreparedModel":
        """The dcut_model record for model_verify: `layers` are dicts as in layer_forward, one paged cache pair per
        layer.  The returned object keeps the tensors alive."""
        L = len(layers)
        assert len(k_caches) == L and len(v_caches) == L
        names = ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")
        lw = (LayerWeights * max(L, 1))(*[LayerWeights(*[_ptr(w[n], torch.bfloat16) for n in names], rms_eps, rope_theta)
                                          for w in layers])
        kc = (_vp * max(L, 1))(*[_ptr(k, torch.bfloat16) for k in k_caches])
        vc = (_vp * max(L, 1))(*[_ptr(v, torch.bfloat16) for v in v_caches])
        rec = Model(L, lw, kc, vc, _ptr(embed, torch.bfloat16), _ptr(g_final, torch.bfloat16), _ptr(w_lm, torch.bfloat16),
                    w_lm.shape[0])
        return PreparedModel(rec, (lw, kc, vc, layers, embed, g_final, w_lm, k_caches, v_caches),
                             k_caches[0].shape[0] if L else 0, embed.device)

    def model_verify(self, model: "PreparedModel", block_table, ctx_lens, cu_q, tok_req, tok_pos, tok_id, draft_ids,
                     T_cap: int, out_tokens: bool = True, row_argmax: bool = False, hidden_out=None, out=None):
        """dcut_model_verify: embedding, the model's decoder layers, final norm, LM head and acceptance in one call.
        `out` = (accept_len, bonus, out_tokens, total, row_argmax) of an earlier call is written in place."""
        B, gamma = draft_ids.shape
        if out is None:
            i32 = dict(dtype=torch.int32, device=model.device)
            out = (torch.empty(B, **i32), torch.empty(B, **i32), torch.empty((B, gamma + 1), **i32) if out_tokens else None,
                   torch.empty(1, **i32), torch.full((T_cap,), -1, **i32) if row_argmax else None)
        accept_len, bonus, toks, total, am = out
        self._check(_lib.dcut_model_verify(self._h, C.byref(model.rec), model.num_pages, _ptr(block_table, torch.int32),
                                           block_table.shape[1], _ptr(ctx_lens, torch.int32), _ptr(cu_q, torch.int32),
                                           _ptr(tok_req, torch.int32), _ptr(tok_pos, torch.int32),
                                           _ptr(tok_id, torch.int32), _ptr(draft_ids, torch.int32), B, gamma, T_cap,
                                           _ptr(accept_len), _ptr(bonus), _ptr(toks), _ptr(total), _ptr(am),
                                           _ptr(hidden_out, torch.bfloat16), _stream()))
        return out

    def poll_device_status(self) -> int:
        code = _i(0)
        st = _lib.dcut_poll_device_status(self._h, C.byref(code), _stream())
        if st not in (OK, EDEVICE):
            self._check(st)
        return code.value
