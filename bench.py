#!/usr/bin/env python
"""Benchmark of the D-cut verify hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl dcut|reference] [--config 2]

A step is one pass of the whole hot path over one batch of synthetic input: dcut_select ->
dcut_verify_attn -> dcut_accept.  The headline value is accepted tokens/s of the D-cut-pruned arm
at B = 64 (workload 2); the full-gamma and gamma = 0 arms, the attention roofline, the end-to-end
number from host buffers and the CPU oracle's throughput ride along in the same JSON line.

`--impl reference` times the CPU oracle (test infrastructure, run as it stands) on a bounded
sample of the same workload.  With N > 1 every rank runs an independent replica of the workload
(the path has no cross-GPU exchange); the value is the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2607_14647_b200 import workloads as wl  # noqa: E402

METRIC = "accepted_tokens_per_s_per_verify_step_B64"
UNIT = "tokens/s"
L2_BYTES = 126e6
# DRAM bytes per algorithmic byte of attn_split_kernel, from the ncu capture on workload 1 summarised under
# profiles/ (1.03 at gamma = 0 to 1.07 at full gamma); the kernel's traffic is proportional to the KV streamed
ATTN_TRAFFIC_RATIO = 1.05


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="dcut", choices=["dcut", "reference"])
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--cost-points", type=int, default=18)
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--gamma", type=int, default=0,
                    help="draft tokens per request, if not the config's (7 = the paper's block-8 setting)")
    ap.add_argument("--layers", type=int, default=0,
                    help="with a layer config (4): time the whole verification forward of a model of this many decoder "
                         "layers (dcut_model_verify) instead of one layer")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch the step's kernels one by one instead of replaying a CUDA graph")
    return ap.parse_args()


# ------------------------------------------------------------------------------------------------ helpers

class ClockSampler:
    """Samples the SM clock and the throttle reasons through NVML (read-only) from a thread while the timed
    region runs; falls back to one nvidia-smi query if NVML is not importable."""
    REASONS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}

    def __init__(self, index: int, period_s: float = 0.005):
        import threading
        self.sm, self.reasons, self.max_mhz, self.index = [], set(), None, index
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            # CUDA_VISIBLE_DEVICES remaps ordinals: find the NVML device by the CUDA device's UUID
            uuid = str(torch.cuda.get_device_properties(index).uuid)
            self._h = None
            for i in range(pynvml.nvmlDeviceGetCount()):
                h = pynvml.nvmlDeviceGetHandleByIndex(i)
                u = pynvml.nvmlDeviceGetUUID(h)
                u = u.decode() if isinstance(u, bytes) else u
                if uuid in u:
                    self._h = h
            if self._h is None:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
            self._thread = threading.Thread(target=self._run, args=(period_s,), daemon=True)
            self._thread.start()
        except Exception:
            self._nv = None

    def _run(self, period_s):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                for name, bit in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(period_s)

    def stop(self) -> dict:
        if self._thread is not None:
            self._stop.set()
            self._thread.join(timeout=2)
        if not self.sm:      # fallback: a single nvidia-smi reading taken now
            try:
                out = subprocess.run(["nvidia-smi", "-i", str(self.index), "--query-gpu=clocks.sm,clocks.max.sm",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=20).stdout
                a, b = out.strip().split(",")
                return {"sm_mhz": float(a), "sm_max_mhz": float(b), "reasons": [], "samples": 1, "source": "nvidia-smi"}
            except Exception:
                return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(self.sm), "sm_min_mhz": min(self.sm), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.sm), "source": "nvml"}


def dist_setup(n_gpus: int):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl" if torch.cuda.is_available() else "gloo")
    return world, rank, local


def max_over_ranks(x: float, world: int) -> float:
    """The slowest rank's value (the only cross-rank exchange of the benchmark)."""
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device="cuda" if dist.get_backend() == "nccl" else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


def attn_algorithmic_bytes(cfg, ctx_lens: np.ndarray, depths: np.ndarray) -> int:
    """K and V of every visible cache position once, Q read, O written, block-table entries."""
    kv_tokens = int((ctx_lens.astype(np.int64) + depths + 1).sum())
    T = int((depths.astype(np.int64) + 1).sum())
    pages = int(((ctx_lens.astype(np.int64) + depths + 1 + cfg.page_size - 1) // cfg.page_size).sum())
    return (kv_tokens * cfg.n_kv_heads * cfg.head_dim * 2 * 2 + 2 * T * cfg.n_q_heads * cfg.head_dim * 2
            + pages * 4 * cfg.n_kv_heads)


def cost_grid(cfg, points: int, tiled: bool) -> list:
    """Packed lengths at which the step is timed for the cost table.  Evenly spaced; where the forward holds GEMMs
    (`tiled`), whose cost moves in steps of their 128-row tiles, the points are the last length of a row block and the
    first of the next, thinned to about `points`, so that the table shows the steps and the selector can stop at them."""
    cap = cfg.t_cap
    if not tiled:
        return sorted(set(int(round(x)) for x in np.linspace(cfg.B, cap, points)))
    edges = [k * 128 for k in range(1, cap // 128 + 1) if cfg.B < k * 128 < cap]
    stride = max(1, int(np.ceil(2 * len(edges) / max(points - 2, 1))))
    pts = {cfg.B, cap}
    for e in edges[::stride]:
        pts.update((e, e + 1))
    return sorted(pts)


def monotone_cost(cost: np.ndarray) -> np.ndarray:
    """Non-decreasing cost table from profiled points.  A longer batch never costs less, so the cost at T is at most
    every measurement at T' >= T: the table is the running minimum taken from the long end.  (A running maximum from
    the short end is monotone too, but one disturbed measurement then lifts every longer entry to its level, and the
    selector, seeing a plateau, runs to the plateau's end.)"""
    return np.minimum.accumulate(np.asarray(cost, np.float64)[::-1])[::-1].astype(np.float32)


def peaks() -> dict:
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------------ CPU oracle legs

def oracle_sample(cfg, sel, kv, q_all, logits_all, cost, seconds: float):
    """Times the oracle, as it stands, on a bounded sample: selection for the whole batch, then
    attention and acceptance request by request until `seconds` of CPU time are used."""
    from oracle import dcut_oracle as orc
    t0 = time.perf_counter()
    r = orc.select(sel.conf, sel.draft_ids, sel.bonus_ids, sel.ctx_lens, cost)
    done, accepted = 0, 0
    for i in range(cfg.B):
        d = int(r.depths[i])
        cu1 = np.array([0, d + 1], np.int32)
        orc.verify_attn(q_all[i, : d + 1].contiguous(), kv.k_cache, kv.v_cache, kv.block_table[i: i + 1],
                        sel.ctx_lens[i: i + 1], cu1, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
        a = orc.accept(logits_all[i, : d + 1].contiguous(), sel.draft_ids[i: i + 1], cu1, cfg.gamma)
        accepted += a.n_accepted_total
        done += 1
        if time.perf_counter() - t0 > seconds:
            break
    dt = time.perf_counter() - t0
    return {"value": accepted / dt, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
            "sample": f"selection for all {cfg.B} requests, attention + acceptance for the first {done} of {cfg.B} "
                      f"requests ({accepted} accepted tokens in {dt:.1f} s)"}, dt, done, accepted


def host_inputs(cfg):
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    full = np.full(cfg.B, cfg.gamma, np.int32)
    q_all = wl.q_rows(cfg, full).view(cfg.B, cfg.gamma + 1, cfg.n_q_heads, cfg.head_dim)
    logits_all = wl.logits_rows(cfg, sel, full).view(cfg.B, cfg.gamma + 1, cfg.vocab)
    return sel, kv, q_all, logits_all


def layer_flops(cfg, T: int) -> float:
    """Dense-projection flops of one layer for T packed tokens (2 * T * parameters)."""
    qkv_w = (cfg.n_q_heads + 2 * cfg.n_kv_heads) * cfg.head_dim
    params = qkv_w * cfg.hidden + cfg.hidden * cfg.n_q_heads * cfg.head_dim + 3 * cfg.intermediate * cfg.hidden
    return 2.0 * T * params


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = wl.config(args.config)
    if args.gamma > 0:
        cfg = dataclasses.replace(cfg, gamma=args.gamma, name=f"{cfg.name}_gamma{args.gamma}")
    sel, kv, q_all, logits_all = host_inputs(cfg)
    cost = wl.cost_table_for(cfg)
    per_step = max(2.0, min(args.cpu_seconds, 120.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_sample(cfg, sel, kv, q_all, logits_all, cost, per_step)
    times, toks, info = [], [], None
    for _ in range(args.steps):
        info, dt, _, acc = oracle_sample(cfg, sel, kv, q_all, logits_all, cost, per_step)
        times.append(dt)
        toks.append(acc)
    value = sum(toks) / sum(times)
    info["value"] = value
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"configs[{cfg.index}] {cfg.name}: B={cfg.B} gamma={cfg.gamma} "
                                   f"{cfg.n_q_heads}q/{cfg.n_kv_heads}kv Dh={cfg.head_dim} V={cfg.vocab}",
                       "cost_table": "linear stand-in (no GPU profile in this arm)"},
            "cpu_baseline": info,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------ GPU arm

def run_dcut(args):
    world, rank, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    from paper_2607_14647_b200 import binding

    cfg = wl.config(args.config)
    if args.gamma > 0:
        cfg = dataclasses.replace(cfg, gamma=args.gamma, name=f"{cfg.name}_gamma{args.gamma}")
    sel, kv, q_all, logits_all = host_inputs(cfg)
    dev = torch.device("cuda", local)
    d_conf = torch.from_numpy(sel.conf).to(dev)
    d_draft = torch.from_numpy(sel.draft_ids).to(dev)
    d_bonus = torch.from_numpy(sel.bonus_ids).to(dev)
    d_ctx = torch.from_numpy(sel.ctx_lens).to(dev)
    d_bt = torch.from_numpy(kv.block_table).to(dev)
    d_k, d_v = kv.k_cache.to(dev), kv.v_cache.to(dev)
    d_q_all = q_all.to(dev).view(cfg.t_cap, cfg.n_q_heads, cfg.head_dim)
    d_logits_all = logits_all.to(dev).view(cfg.t_cap, cfg.vocab)
    is_layer = cfg.hidden > 0
    ctx = binding.Context(max_B=cfg.B, max_gamma=cfg.gamma, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
                          head_dim=cfg.head_dim, page_size=cfg.page_size, max_pages_per_req=kv.max_pages_per_req,
                          vocab=cfg.vocab, hidden=cfg.hidden, intermediate=cfg.intermediate)
    cap = cfg.t_cap
    sel_out = None
    if is_layer:
        lw = wl.layer_weights(cfg)
        d_w = {n: getattr(lw, n).to(dev) for n in ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")}
        d_x_all = wl.layer_x_rows(cfg, np.full(cfg.B, cfg.gamma, np.int32)).to(dev)

    def pack(depths_np):
        """Gathers the kept rows (i, t <= d_i) of the unpacked device tensors (set-up, not timed)."""
        idx = np.concatenate([i * (cfg.gamma + 1) + np.arange(d + 1) for i, d in enumerate(depths_np)])
        idx_t = torch.from_numpy(idx).to(dev)
        first = d_x_all if is_layer else d_q_all
        return first.index_select(0, idx_t).contiguous(), d_logits_all.index_select(0, idx_t).contiguous()

    res = {}

    def middle(qp, so, bufs):
        """The verification forward between selection and acceptance: attention, or the whole decoder layer."""
        if is_layer:
            ctx.layer_forward(d_w, qp, bufs["attn_out"], d_k, d_v, d_bt, d_ctx, so.cu_q, so.tok_req, so.tok_pos, cap,
                              cfg.rms_eps, cfg.rope_theta)
        else:
            ctx.verify_attn(qp, d_k, d_v, d_bt, d_ctx, so.cu_q, cap, out=bufs["attn_out"])

    def step(qp, lp, bufs):
        nonlocal sel_out
        sel_out = ctx.select(d_conf, d_draft, d_bonus, d_ctx, out=sel_out)
        middle(qp, sel_out, bufs)
        ctx.accept_into(lp, d_draft, sel_out.cu_q, cap, bufs["accept_len"], bufs["bonus"], bufs["out_tokens"],
                        bufs["total"])

    def make_bufs(T):
        i32 = dict(dtype=torch.int32, device=dev)
        mid = (T, cfg.hidden) if is_layer else (T, cfg.n_q_heads, cfg.head_dim)
        return dict(attn_out=torch.empty(mid, dtype=torch.bfloat16, device=dev),
                    accept_len=torch.empty(cfg.B, **i32), bonus=torch.empty(cfg.B, **i32),
                    out_tokens=torch.empty((cfg.B, cfg.gamma + 1), **i32), total=torch.empty(1, **i32))

    def depths_now():
        step_sel = ctx.select(d_conf, d_draft, d_bonus, d_ctx)
        torch.cuda.synchronize()
        return step_sel.depths.cpu().numpy()

    # ---- cost table: step latency against the packed length T, profiled on this GPU ---------------
    grid = cost_grid(cfg, args.cost_points, is_layer)
    prof = []
    for T in grid:
        ctx.set_cost_buckets(cfg.B, cfg.gamma, [T], [1.0])
        d = depths_now()
        qp, lp = pack(d)
        bufs = make_bufs(T)
        for _ in range(3):
            step(qp, lp, bufs)
        ts = []
        for _ in range(11):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            step(qp, lp, bufs)
            e1.record()
            e1.synchronize()
            ts.append(e0.elapsed_time(e1))
        prof.append(float(np.percentile(ts, 25)))   # interference only ever adds time: lean on the fast side of the sample
        del qp, lp, bufs
    cost = np.interp(np.arange(cap + 1), grid, prof)
    cost = monotone_cost(cost)

    arms = {"pruned": cost, "full_gamma": np.ones(cap + 1, np.float32),
            "gamma0": (1.0 + 10.0 * np.maximum(0, np.arange(cap + 1) - cfg.B)).astype(np.float32)}
    sampler = ClockSampler(local) if rank == 0 else None
    for name, table in arms.items():
        ctx.set_cost_dense(table)
        d = depths_now()
        qp, lp = pack(d)
        T = int(d.sum()) + cfg.B
        bufs = make_bufs(T)
        for _ in range(max(3, args.warmup)):
            step(qp, lp, bufs)
        # (a) kernel-by-kernel launches, with events around the verification forward (attention roofline)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        barrier(world)
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        for k in range(args.steps):
            nonlocal_sel = ctx.select(d_conf, d_draft, d_bonus, d_ctx, out=sel_out)
            ev[k][0].record()
            middle(qp, nonlocal_sel, bufs)
            ev[k][1].record()
            ctx.accept_into(lp, d_draft, nonlocal_sel.cu_q, cap, bufs["accept_len"], bufs["bonus"],
                            bufs["out_tokens"], bufs["total"])
        end.record()
        barrier(world)
        eager_ms = max_over_ranks(start.elapsed_time(end), world)
        attn_ms = statistics.mean(a.elapsed_time(b) for a, b in ev)
        total_ms = eager_ms
        # (b) the same step captured once in a CUDA graph and replayed: the packed length is read on the device,
        # so one graph serves whatever depth vector the selector produces
        if not args.no_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step(qp, lp, bufs)
            for _ in range(3):
                graph.replay()
            barrier(world)
            start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            start.record()
            for k in range(args.steps):
                graph.replay()
            end.record()
            barrier(world)
            total_ms = max_over_ranks(start.elapsed_time(end), world)
            del graph
        accepted = int(bufs["total"].item())
        assert ctx.poll_device_status() == 0
        res[name] = dict(T=T, accepted=accepted, ms_per_step=total_ms / args.steps, eager_ms=eager_ms / args.steps, attn_ms=attn_ms,
                         tokens_per_s=world * accepted / (total_ms / args.steps * 1e-3),
                         attn_bytes=attn_algorithmic_bytes(cfg, sel.ctx_lens, d), depths=d)
        del qp, lp, bufs
    clocks = sampler.stop() if sampler else {}

    # ---- end to end from host buffers ---------------------------------------------------------
    ctx.set_cost_dense(cost)
    e2e = None
    if not is_layer:
        pin = lambda t: t.contiguous().pin_memory()
        h = dict(conf=pin(torch.from_numpy(sel.conf)), draft=pin(torch.from_numpy(sel.draft_ids)),
                 bonus=pin(torch.from_numpy(sel.bonus_ids)), ctx=pin(torch.from_numpy(sel.ctx_lens)),
                 bt=pin(torch.from_numpy(kv.block_table)), q=pin(q_all), logits=pin(logits_all))
        hout = ctx.host_step_outputs(cfg.B, cfg.gamma)
        call = lambda: ctx.verify_step_host(h["conf"], h["draft"], h["bonus"], h["ctx"], h["bt"], h["q"], h["logits"],
                                            d_k, d_v, out=hout)
        for _ in range(3):
            call()
        barrier(world)
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            call()
        barrier(world)
        e2e_s = max_over_ranks(time.perf_counter() - t0, world) / args.e2e_steps
        e2e_accepted = int(hout["n_accepted_total"].item())
        assert e2e_accepted == res["pruned"]["accepted"], (e2e_accepted, res["pruned"]["accepted"])
        e2e = {"value": world * e2e_accepted / e2e_s, "unit": UNIT, "ms_per_step": round(e2e_s * 1e3, 4),
               "h2d_bytes_per_step": hout["h2d_bytes"], "d2h_bytes_per_step": hout["d2h_bytes"],
               "api": "dcut_verify_step_host (pinned host buffers; KV cache resident)"}

    # ---- the four projections of the layer, timed alone (tensor roofline) ---------------------------
    gemm = None
    if is_layer and rank == 0:
        gemm = {}
        qkv_w, q_w = (cfg.n_q_heads + 2 * cfg.n_kv_heads) * cfg.head_dim, cfg.n_q_heads * cfg.head_dim
        for arm in ("pruned", "full_gamma"):
            T = res[arm]["T"]
            cu1 = torch.tensor([0, T], dtype=torch.int32, device=dev)
            rows = {}
            for name, (w, w2, mode, K, N) in {"qkv": (d_w["w_qkv"], None, 0, cfg.hidden, qkv_w),
                                              "o": (d_w["w_o"], None, 1, q_w, cfg.hidden),
                                              "gate_up_swiglu": (d_w["w_gate"], d_w["w_up"], 2, cfg.hidden, cfg.intermediate),
                                              "down": (d_w["w_down"], None, 1, cfg.intermediate, cfg.hidden)}.items():
                a_in = torch.randn((cap, K), device=dev, dtype=torch.float32).to(torch.bfloat16)
                outb = torch.empty((cap, N), dtype=torch.bfloat16, device=dev)
                resb = torch.zeros((cap, N), dtype=torch.bfloat16, device=dev) if mode == 1 else None
                for _ in range(3):
                    ctx.gemm_bf16(a_in, w, cu1, cap, outb, mode=mode, w2=w2, residual=resb)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(20):
                    ctx.gemm_bf16(a_in, w, cu1, cap, outb, mode=mode, w2=w2, residual=resb)
                e1.record()
                e1.synchronize()
                ms = e0.elapsed_time(e1) / 20
                fl = 2.0 * T * K * N * (2 if mode == 2 else 1)
                rows[name] = {"ms": round(ms, 4), "tflops": round(fl / ms / 1e9, 1)}
            tot_ms = sum(r["ms"] for r in rows.values())
            rows["all"] = {"ms": round(tot_ms, 4), "tflops": round(layer_flops(cfg, T) / tot_ms / 1e9, 1)}
            gemm[arm] = rows
        # LM head fused with acceptance (logits never stored) beside the unfused pair, full-gamma packing
        try:
            V = cfg.vocab
            Vp = (V + 255) // 256 * 256
            T = res["full_gamma"]["T"]
            cu_full = torch.arange(0, cfg.B + 1, dtype=torch.int32, device=dev) * (cfg.gamma + 1)
            w_lm = torch.zeros((Vp, cfg.hidden), dtype=torch.bfloat16, device=dev)
            w_lm[:V] = wl.lm_head_weight(cfg).to(dev)
            xh = torch.randn((cap, cfg.hidden), device=dev, dtype=torch.float32).to(torch.bfloat16)
            logits_buf = torch.empty((cap, Vp), dtype=torch.bfloat16, device=dev)

            def timed(fn, n=10):
                for _ in range(2):
                    fn()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(n):
                    fn()
                e1.record()
                e1.synchronize()
                return e0.elapsed_time(e1) / n

            fused_ms = timed(lambda: ctx.lm_head_accept(xh, w_lm[:V], d_draft, cu_full, cap, out_tokens=False))
            gemm_ms = timed(lambda: ctx.gemm_bf16(xh, w_lm, cu_full, cap, logits_buf))
            ctx_v = binding.Context(max_B=cfg.B, max_gamma=cfg.gamma, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
                                    head_dim=cfg.head_dim, page_size=cfg.page_size, max_pages_per_req=1, vocab=Vp)
            acc_ms = timed(lambda: ctx_v.accept(logits_buf, d_draft, cu_full, cap, out_tokens=False))
            fl = 2.0 * T * cfg.hidden * V
            gemm["lm_head"] = {"T": T, "V": V, "fused_ms": round(fused_ms, 4), "fused_tflops": round(fl / fused_ms / 1e9, 1),
                               "unfused_gemm_ms": round(gemm_ms, 4), "unfused_accept_ms": round(acc_ms, 4),
                               "logits_bytes_not_moved": 2 * T * V * 2}
            del w_lm, logits_buf, ctx_v
        except Exception as exc:   # the extra measurement must not take the bench line down
            gemm["lm_head"] = {"error": repr(exc)[:200]}

    # ---- stochastic variant (causal selector + rejection-sampling acceptance), timed alone at full depth ----------
    stochastic = None
    if not is_layer and rank == 0:
        try:
            def timed_us(fn, n=20):
                for _ in range(3):
                    fn()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(n):
                    fn()
                e1.record()
                e1.synchronize()
                return e0.elapsed_time(e1) / n * 1e3

            ctx.set_cost_dense(cost)
            t_sel = timed_us(lambda: ctx.select(d_conf, d_draft, d_bonus, d_ctx, out=sel_out))
            t_selc = timed_us(lambda: ctx.select(d_conf, d_draft, d_bonus, d_ctx, out=sel_out, causal=True))
            full = np.full(cfg.B, cfg.gamma, np.int32)
            cu_full = torch.from_numpy(wl.cu_q_from_depths(full)).to(dev)
            # drafter logits: the target rows plus noise (generated on the device; the values do not change the traffic)
            idx = torch.from_numpy(np.concatenate([i * (cfg.gamma + 1) + np.arange(cfg.gamma) for i in range(cfg.B)])).to(dev)
            d_dl = d_logits_all.index_select(0, idx).view(cfg.B, cfg.gamma, cfg.vocab).contiguous()
            d_dl += (0.3 * torch.randn(d_dl.shape, device=dev, dtype=torch.float32)).to(torch.bfloat16)
            ua_np, us_np = wl.uniforms(cfg)
            d_ua, d_us = torch.from_numpy(ua_np).to(dev), torch.from_numpy(us_np).to(dev)
            dr = (d_draft % cfg.vocab).contiguous()
            t_rs = timed_us(lambda: ctx.accept_rs(d_logits_all, d_dl, dr, cu_full, cap, d_ua, d_us), n=10)
            rs_bytes = 2 * cfg.vocab * (cfg.t_cap + cfg.B * cfg.gamma)
            stochastic = {"select_us": round(t_sel, 2), "select_causal_us": round(t_selc, 2),
                          "accept_rs_us": round(t_rs, 1), "accept_rs_scan_bytes": rs_bytes,
                          "accept_rs_gbs": round(rs_bytes / (t_rs * 1e-6) / 1e9, 1)}
            del d_dl
        except Exception as exc:   # the extra measurement must not take the bench line down
            stochastic = {"error": repr(exc)[:200]}

    if rank != 0:
        return
    pk = peaks()
    p = res["pruned"]
    achieved = p["attn_bytes"] / (p["attn_ms"] * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": p["tokens_per_s"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": p["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"configs[{cfg.index}] {cfg.name}: B={cfg.B} gamma={cfg.gamma} {cfg.n_q_heads}q/"
                               f"{cfg.n_kv_heads}kv Dh={cfg.head_dim} page={cfg.page_size} V={cfg.vocab} "
                               f"ctx {cfg.ctx_lo}-{cfg.ctx_hi}",
                   "arm": "D-cut pruned (dense cost table profiled on this GPU)",
                   "launch": "kernel by kernel" if args.no_graph else "one CUDA graph of the step, replayed each step",
                   "l2": f"inputs exceed L2: each step streams {p['attn_bytes'] / 1e6:.0f} MB of KV and "
                         f"{p['T'] * cfg.vocab * 2 / 1e6:.0f} MB of logits once (L2 is 126 MB)",
                   "parallelism": "replicas only" if world > 1 else "1 GPU"},
        "arms": {k: {"T": v["T"], "accepted_tokens": v["accepted"], "ms_per_step": round(v["ms_per_step"], 4),
                     "ms_per_step_kernel_by_kernel": round(v["eager_ms"], 4),
                     "attn_ms": round(v["attn_ms"], 4), "tokens_per_s": round(v["tokens_per_s"], 1),
                     "attn_gbs": round(v["attn_bytes"] / (v["attn_ms"] * 1e-3) / 1e9, 1)} for k, v in res.items()},
        "roofline": {"kernel": "dcut_verify_attn (attn_plan_kernel + attn_item_kernel + attn_combine_kernel)", "bound": "hbm",
                     "achieved": round(achieved, 1), "peak": pk["hbm_gbs"], "unit": "GB/s",
                     "frac": round(achieved / pk["hbm_gbs"], 4), "peak_source": f"of {pk['source']}",
                     "frac_of_8000_nominal": round(achieved / 8000.0, 4),
                     "algorithmic_bytes_per_launch": p["attn_bytes"],
                     "traffic": None if ATTN_TRAFFIC_RATIO is None else int(ATTN_TRAFFIC_RATIO * p["attn_bytes"])},
        "e2e": e2e,
        "gpu_launches": (14 if is_layer else 6) * args.steps,
        "cost_table_ms": {str(t): round(c, 4) for t, c in zip(grid, prof)},
        "clocks": clocks,
    }
    if stochastic is not None:
        line["stochastic"] = stochastic
    if is_layer:
        pkj = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")) else {}
        tf_peak = float(pkj.get("bf16_tflops", 1590.0))
        line["config"]["arm"] += "; verification forward = one decoder layer (dcut_layer_forward)"
        line["layer"] = {"gemm_alone": gemm, "flops_per_token": layer_flops(cfg, 1)}
        g = gemm["full_gamma"]["all"]
        for v in line["arms"].values():   # here the timed middle stage is the whole layer, not attention alone
            v["forward_ms"] = v.pop("attn_ms")
            v.pop("attn_gbs")
        line["roofline"] = line["roofline_tensor"] = {"kernel": "gemm_tcgen05_kernel (4 projections of the layer, full-gamma arm, timed alone)",
                                   "bound": "tensor", "achieved": g["tflops"], "peak": tf_peak, "unit": "TFLOP/s",
                                   "frac": round(g["tflops"] / tf_peak, 4),
                                   "peak_source": "of measured (burst)" if pkj else "of fallback", "traffic": None}
    if world == 1 and not args.no_cpu_baseline and not is_layer:
        info, *_ = oracle_sample(cfg, sel, kv, q_all, logits_all, cost, args.cpu_seconds)
        line["cpu_baseline"] = info
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------ whole-model arm

def run_model(args):
    """select -> dcut_model_verify (embedding, L layers, final norm, LM head + acceptance) per step, for a random-init
    model of the layer config's shapes.  Weights and the per-layer KV caches are drawn on the device (seeded)."""
    world, rank, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    from paper_2607_14647_b200 import binding
    cfg = wl.config(args.config)
    if cfg.hidden <= 0:
        raise SystemExit("--layers needs a layer config (--config 4)")
    L, H, I, V = args.layers, cfg.hidden, cfg.intermediate, cfg.vocab
    dev = torch.device("cuda", local)
    sel = wl.select_inputs(cfg)
    kv = wl.paged_kv(cfg, sel.ctx_lens)
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.seed)

    def w(r, c, scale=0.02):
        return (torch.randn((r, c), generator=gen, device=dev, dtype=torch.float32) * scale).to(torch.bfloat16)

    qkv_rows, q_w = (cfg.n_q_heads + 2 * cfg.n_kv_heads) * cfg.head_dim, cfg.n_q_heads * cfg.head_dim
    ones = torch.ones(H, dtype=torch.bfloat16, device=dev)
    layers = [dict(w_qkv=w(qkv_rows, H), w_o=w(H, q_w), w_gate=w(I, H), w_up=w(I, H), w_down=w(H, I), g_attn=ones, g_mlp=ones)
              for _ in range(L)]
    k0, v0 = kv.k_cache.to(dev), kv.v_cache.to(dev)
    k_caches = [k0] + [k0.clone() for _ in range(L - 1)]       # own memory per layer; the contents do not matter for time
    v_caches = [v0] + [v0.clone() for _ in range(L - 1)]
    embed, w_lm = w(V, H, 1.0), w(V, H)
    d_conf, d_draft = torch.from_numpy(sel.conf).to(dev), torch.from_numpy(sel.draft_ids % V).to(dev)
    d_bonus, d_ctx = torch.from_numpy(sel.bonus_ids % V).to(dev), torch.from_numpy(sel.ctx_lens).to(dev)
    d_bt = torch.from_numpy(kv.block_table).to(dev)
    ctx = binding.Context(max_B=cfg.B, max_gamma=cfg.gamma, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
                          head_dim=cfg.head_dim, page_size=cfg.page_size, max_pages_per_req=kv.max_pages_per_req,
                          vocab=V, hidden=H, intermediate=I)
    model = ctx.make_model(layers, embed, ones, w_lm, k_caches, v_caches, cfg.rms_eps, cfg.rope_theta)
    cap = cfg.t_cap
    state = {"sel": None, "out": None}

    def step(ev=None):
        so = state["sel"] = ctx.select(d_conf, d_draft, d_bonus, d_ctx, out=state["sel"])
        if ev:
            ev[0].record()
        state["out"] = ctx.model_verify(model, d_bt, d_ctx, so.cu_q, so.tok_req, so.tok_pos, so.tok_id, d_draft, cap,
                                        out=state["out"])
        if ev:
            ev[1].record()

    def timed(n):
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        barrier(world)
        start.record()
        for k in range(n):
            step(evs[k])
        end.record()
        barrier(world)
        return max_over_ranks(start.elapsed_time(end), world) / n, statistics.mean(a.elapsed_time(b) for a, b in evs)

    def depths_now():
        so = ctx.select(d_conf, d_draft, d_bonus, d_ctx)
        torch.cuda.synchronize()
        return so.depths.cpu().numpy()

    grid = cost_grid(cfg, args.cost_points, True)
    prof = []
    for T in grid:                                   # step latency against the packed length, profiled on this GPU
        ctx.set_cost_buckets(cfg.B, cfg.gamma, [T], [1.0])
        step()
        prof.append(timed(3)[0])
    cost = monotone_cost(np.interp(np.arange(cap + 1), grid, prof))
    arms = {"pruned": cost, "full_gamma": np.ones(cap + 1, np.float32),
            "gamma0": (1.0 + 10.0 * np.maximum(0, np.arange(cap + 1) - cfg.B)).astype(np.float32)}
    flops_tok = L * layer_flops(cfg, 1) + 2.0 * H * V
    res = {}
    sampler = ClockSampler(local) if rank == 0 else None
    for name, table in arms.items():
        ctx.set_cost_dense(table)
        d = depths_now()
        T = int(d.sum()) + cfg.B
        for _ in range(max(3, args.warmup)):
            step()
        eager_ms, fwd_ms = timed(args.steps)
        ms = eager_ms
        if not args.no_graph:
            # the same step captured once in a CUDA graph and replayed (the packed length is read on the device)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            for _ in range(3):
                graph.replay()
            barrier(world)
            start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            start.record()
            for _ in range(args.steps):
                graph.replay()
            end.record()
            barrier(world)
            ms = max_over_ranks(start.elapsed_time(end), world) / args.steps
            del graph
        assert ctx.poll_device_status() == 0
        planted = int((np.minimum(d, sel.reject_index) + 1).sum())
        res[name] = {"T": T, "ms_per_step": round(ms, 4), "ms_per_step_kernel_by_kernel": round(eager_ms, 4), "forward_ms": round(fwd_ms, 4),
                     "accepted_tokens_planted": planted, "accepted_tokens_by_the_random_init_model": int(state["out"][3].item()),
                     "tokens_per_s": round(world * planted / (ms * 1e-3), 1),
                     "verified_tokens_per_s": round(world * T / (ms * 1e-3), 1),
                     "forward_tflops": round(flops_tok * T / fwd_ms / 1e9, 1),
                     "kv_streamed_gb": round(L * attn_algorithmic_bytes(cfg, sel.ctx_lens, d) / 1e9, 2)}
    clocks = sampler.stop() if sampler else {}
    if rank != 0:
        return
    pkj = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")) else {}
    tf_peak = float(pkj.get("bf16_tflops_sustained", pkj.get("bf16_tflops", 1400.0)))
    p = res["pruned"]
    weights_gb = (L * (qkv_rows * H + H * q_w + 3 * H * I) + 2 * V * H) * 2 / 1e9
    line = {
        "metric": METRIC, "value": p["tokens_per_s"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
        "ms_per_step": p["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": f"configs[{cfg.index}] {cfg.name} as a {L}-layer model: B={cfg.B} gamma={cfg.gamma} {cfg.n_q_heads}q/"
                               f"{cfg.n_kv_heads}kv Dh={cfg.head_dim} hidden={H} intermediate={I} V={V} ctx {cfg.ctx_lo}-{cfg.ctx_hi}",
                   "arm": "D-cut pruned (cost table profiled on this GPU); step = dcut_select + dcut_model_verify",
                   "accepted_tokens": "random-init weights accept no draft, so the numerator is the workload's planted acceptance "
                                      "min(d_i, reject_index_i) + 1 per request; the LM head, argmax and prefix match run in the timed region",
                   "launch": "kernel by kernel (programmatic dependent launch)" if args.no_graph else "one CUDA graph of the step, replayed each step",
                   "l2": f"each step streams {weights_gb:.1f} GB of weights and {p['kv_streamed_gb']:.1f} GB of KV once (L2 is 126 MB)",
                   "parallelism": "replicas only" if world > 1 else "1 GPU"},
        "arms": res,
        "roofline": {"kernel": "all kernels of dcut_model_verify (projections, attention, norms, LM head), pruned arm",
                     "bound": "tensor", "achieved": p["forward_tflops"], "peak": tf_peak, "unit": "TFLOP/s",
                     "frac": round(p["forward_tflops"] / tf_peak, 4),
                     "peak_source": "of measured (sustained)" if "bf16_tflops_sustained" in pkj else "of fallback", "traffic": None},
        "e2e": None, "gpu_launches": (5 + 10 * L) * args.steps,   # select, embed, 10 per layer, norm, LM head, match
        "cost_table_ms": {str(t): round(c, 4) for t, c in zip(grid, prof)}, "clocks": clocks,
    }
    print(json.dumps(line))


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.layers > 0:
        run_model(args)
    else:
        run_dcut(args)


if __name__ == "__main__":
    main()
