#!/usr/bin/env python
"""Benchmark of the D-cut verify hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl dcut|reference] [--config 2]

A step is one pass of the whole hot path over one batch of synthetic input: dcut_select ->
dcut_verify_attn -> dcut_accept (for the layer workload: the whole decoder layer in the middle).
The headline value is accepted tokens/s of the D-cut-pruned arm at B = 64 (workload 2); the
full-gamma, gamma = 0 and paper-bucket arms, the attention roofline, the end-to-end number from
host buffers, the CPU oracle's throughput and bounded runs of workloads 1, 3 and 4 ride along in
the same JSON line.

Timing: every arm is warmed up (>= 20 steps), then its CUDA graph is replayed `--steps` times
between a barrier + synchronize on both sides, and that loop is repeated until at least 100 steps
and 0.5 s have been timed; `ms_per_step` is the mean over all of them, and a second pass with an
event after every replay gives the median and the 95th percentile per step.

`--impl reference` times the CPU oracle (test infrastructure, run as it stands) on a bounded
sample of the same workload.  With N > 1 every rank runs an independent replica of the workload
(the path has no cross-GPU exchange); the value is the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import math
import os
import statistics
import subprocess
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2607_14647_b200 import workloads as wl  # noqa: E402

METRIC = "accepted_tokens_per_s_per_verify_step_B64"
UNIT = "tokens/s"
L2_BYTES = 126e6
# DRAM bytes per algorithmic byte of attn_item_kernel, from ncu captures (dram__bytes_read.sum + dram__bytes_write.sum of
# one launch) summarised in profiles/attn_item_kernel_dram_traffic.md: 1.001-1.005 over the three arms of workload 2 at
# full size and of workload 3's shapes at B = 48; the kernel's traffic is proportional to the KV it streams
ATTN_TRAFFIC_RATIO = 1.004
RATIO_BUCKETS = [(1, 4), (1, 2), (3, 4), (1, 1)]          # the paper's ratio set R (Eq. 4; Table 3)
COST_INNER = 4        # steps per timed sample of the cost profile (CUDA event stamps step by 1-2 us)
COST_PROFILE_DIR = os.path.join(ROOT, "paper_2607_14647_b200", "cost_profiles")


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="dcut", choices=["dcut", "reference"])
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--cost-points", type=int, default=18)
    ap.add_argument("--cost-reps", type=int, default=15, help="replays per cost-table point (their median is the point)")
    ap.add_argument("--min-timed-steps", type=int, default=100)
    ap.add_argument("--min-timed-seconds", type=float, default=0.5)
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--gamma", type=int, default=0,
                    help="draft tokens per request, if not the config's (7 = the paper's block-8 setting)")
    ap.add_argument("--layers", type=int, default=0,
                    help="with a layer config (4): time the whole verification forward of a model of this many decoder "
                         "layers (dcut_model_verify) instead of one layer")
    ap.add_argument("--extras", default="auto",
                    help="bounded runs of other workloads on the same line: 'auto' (1,3,4 beside the default workload 2 on "
                         "one GPU), 'none', or a comma list of config indices")
    ap.add_argument("--multistep", type=int, default=8, help="steps chained on the device (select..commit) in the multi-step arm; 0: skip")
    ap.add_argument("--attn-only", action="store_true",
                    help="run only dcut_verify_attn, `--steps` launches per arm after `--warmup` (the command ncu captures)")
    ap.add_argument("--batch", type=int, default=0, help="with --attn-only: this many requests instead of the config's B (small ncu captures)")
    ap.add_argument("--write-cost-profile", action="store_true",
                    help="store the profiled cost points under paper_2607_14647_b200/cost_profiles/ (read by --impl reference)")
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
        self.t0 = time.perf_counter()
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
        span = time.perf_counter() - self.t0
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
                "reasons": sorted(self.reasons), "samples": len(self.sm), "sampled_seconds": round(span, 3), "source": "nvml"}


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
    """Non-decreasing cost table by a running minimum from the long end (a measurement at T' bounds the cost at every
    T <= T').  Kept for the layer workloads, whose cost moves in steps that an averaging fit would smear."""
    return np.minimum.accumulate(np.asarray(cost, np.float64)[::-1])[::-1].astype(np.float32)


def peaks() -> dict:
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def stats_ms(samples) -> dict:
    a = np.asarray(samples, np.float64)
    return {"median": round(float(np.median(a)), 4), "p95": round(float(np.percentile(a, 95)), 4), "n": int(len(a))}


def workload_name(cfg) -> str:
    s = (f"configs[{cfg.index}] {cfg.name}: B={cfg.B} gamma={cfg.gamma} {cfg.n_q_heads}q/{cfg.n_kv_heads}kv "
         f"Dh={cfg.head_dim} page={cfg.page_size} V={cfg.vocab} ctx {cfg.ctx_lo}-{cfg.ctx_hi}")
    if cfg.hidden > 0:
        s += f" hidden={cfg.hidden} intermediate={cfg.intermediate}"
    return s


COST_TABLE_NOTE = ("dense in the packed length T: step latency profiled on B200 (median of graph replays per point, "
                   "isotonic fit, linear interpolation)")


def stored_cost_profile(cfg):
    """Cost points of an earlier bench.py --write-cost-profile run on a B200 of this pool, or None."""
    p = os.path.join(COST_PROFILE_DIR, f"b200_config{cfg.index}_gamma{cfg.gamma}.json")
    if not os.path.exists(p):
        return None
    d = json.load(open(p))
    return d if d.get("B") == cfg.B and d.get("gamma") == cfg.gamma else None


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
            "sample": f"selection for all {cfg.B} requests (T = {r.t_total}), attention + acceptance for the first {done} of "
                      f"{cfg.B} requests ({accepted} accepted tokens in {dt:.1f} s)"}, dt, done, accepted


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
    from paper_2607_14647_b200 import profiler
    cfg = wl.config(args.config)
    if args.gamma > 0:
        cfg = dataclasses.replace(cfg, gamma=args.gamma, name=f"{cfg.name}_gamma{args.gamma}")
    sel, kv, q_all, logits_all = host_inputs(cfg)
    stored = stored_cost_profile(cfg)
    if stored is not None:
        # the same table the GPU arm's selector reads, up to the noise between two profiling runs of one protocol
        cost = profiler.dense_table(stored["T"], stored["median_ms"], cfg.t_cap + 1)
        source = "stored B200 profile (" + os.path.relpath(COST_PROFILE_DIR, ROOT) + ")"
    else:
        cost = wl.cost_table_for(cfg)
        source = "linear stand-in (no stored B200 profile for this workload)"
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
            "config": {"workload": workload_name(cfg), "arm": "D-cut pruned", "cost_table": COST_TABLE_NOTE},
            "cost_table_source": source,
            "cpu_baseline": info,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------ GPU arm

class Workload:
    """One workload resident on the GPU: inputs, context, the step, its graphs."""

    def __init__(self, cfg, dev, kv_copies: int = 0, spare_pages: int = 0):
        from paper_2607_14647_b200 import binding
        self.cfg, self.dev = cfg, dev
        self.sel, self.kv, q_all, logits_all = host_inputs(cfg) if spare_pages == 0 else self._inputs_with_spares(cfg, spare_pages)
        self.q_all_host, self.logits_all_host = q_all, logits_all
        sel, kv = self.sel, self.kv
        self.is_layer = cfg.hidden > 0
        t = torch.from_numpy
        self.d_conf, self.d_draft = t(sel.conf).to(dev), t(sel.draft_ids).to(dev)
        self.d_bonus, self.d_ctx, self.d_bt = t(sel.bonus_ids).to(dev), t(sel.ctx_lens).to(dev), t(kv.block_table).to(dev)
        # L2 honesty: when one pass over the KV does not dwarf the 126 MB L2, consecutive steps rotate over independent
        # copies of the cache, so that no step finds the previous step's lines resident
        kv_bytes = 2 * kv.k_cache.numel() * 2
        if kv_copies == 0:
            kv_copies = 3 if kv_bytes < 4 * L2_BYTES else 1
        self.kv_copies = kv_copies
        k0, v0 = kv.k_cache.to(dev), kv.v_cache.to(dev)
        self.d_k = [k0] + [k0.clone() for _ in range(kv_copies - 1)]
        self.d_v = [v0] + [v0.clone() for _ in range(kv_copies - 1)]
        self.d_q_all = q_all.to(dev).view(cfg.t_cap, cfg.n_q_heads, cfg.head_dim)
        self.d_logits_all = logits_all.to(dev).view(cfg.t_cap, cfg.vocab)
        self.ctx = binding.Context(max_B=cfg.B, max_gamma=cfg.gamma, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
                                   head_dim=cfg.head_dim, page_size=cfg.page_size, max_pages_per_req=kv.block_table.shape[1],
                                   vocab=cfg.vocab, hidden=cfg.hidden, intermediate=cfg.intermediate)
        self.ctx.enable_plan_in_select(True)     # the selector leaves the attention work list ready: one launch fewer per step
        self.cap = cfg.t_cap
        self.sel_out = None
        if self.is_layer:
            lw = wl.layer_weights(cfg)
            self.d_w = {n: getattr(lw, n).to(dev) for n in ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")}
            self.d_x_all = wl.layer_x_rows(cfg, np.full(cfg.B, cfg.gamma, np.int32)).to(dev)

    @staticmethod
    def _inputs_with_spares(cfg, spare_pages):
        sel = wl.select_inputs(cfg)
        kv = wl.paged_kv(cfg, sel.ctx_lens, extra_pages=spare_pages)
        full = np.full(cfg.B, cfg.gamma, np.int32)
        q_all = wl.q_rows(cfg, full).view(cfg.B, cfg.gamma + 1, cfg.n_q_heads, cfg.head_dim)
        logits_all = wl.logits_rows(cfg, sel, full).view(cfg.B, cfg.gamma + 1, cfg.vocab)
        return sel, kv, q_all, logits_all

    def close(self):
        self.ctx.close()

    # ---- pieces of the step
    def pack(self, depths_np):
        """Gathers the kept rows (i, t <= d_i) of the unpacked device tensors (set-up, not timed)."""
        cfg = self.cfg
        idx = np.concatenate([i * (cfg.gamma + 1) + np.arange(d + 1) for i, d in enumerate(depths_np)])
        idx_t = torch.from_numpy(idx).to(self.dev)
        first = self.d_x_all if self.is_layer else self.d_q_all
        return first.index_select(0, idx_t).contiguous(), self.d_logits_all.index_select(0, idx_t).contiguous()

    def make_bufs(self, T):
        cfg = self.cfg
        i32 = dict(dtype=torch.int32, device=self.dev)
        mid = (T, cfg.hidden) if self.is_layer else (T, cfg.n_q_heads, cfg.head_dim)
        return dict(attn_out=torch.empty(mid, dtype=torch.bfloat16, device=self.dev),
                    accept_len=torch.empty(cfg.B, **i32), bonus=torch.empty(cfg.B, **i32),
                    out_tokens=torch.empty((cfg.B, cfg.gamma + 1), **i32), total=torch.empty(1, **i32))

    def select(self):
        self.sel_out = self.ctx.select(self.d_conf, self.d_draft, self.d_bonus, self.d_ctx, out=self.sel_out)
        return self.sel_out

    def middle(self, qp, so, bufs, copy=0):
        """The verification forward between selection and acceptance: attention, or the whole decoder layer."""
        cfg = self.cfg
        if self.is_layer:
            self.ctx.layer_forward(self.d_w, qp, bufs["attn_out"], self.d_k[copy], self.d_v[copy], self.d_bt, self.d_ctx,
                                   so.cu_q, so.tok_req, so.tok_pos, self.cap, cfg.rms_eps, cfg.rope_theta)
        else:
            self.ctx.verify_attn(qp, self.d_k[copy], self.d_v[copy], self.d_bt, self.d_ctx, so.cu_q, self.cap, out=bufs["attn_out"])

    def accept(self, lp, so, bufs):
        self.ctx.accept_into(lp, self.d_draft, so.cu_q, self.cap, bufs["accept_len"], bufs["bonus"], bufs["out_tokens"],
                             bufs["total"])

    def step(self, qp, lp, bufs, copy=0):
        so = self.select()
        self.middle(qp, so, bufs, copy)
        self.accept(lp, so, bufs)

    def depths_now(self):
        so = self.ctx.select(self.d_conf, self.d_draft, self.d_bonus, self.d_ctx)
        torch.cuda.synchronize()
        return so.depths.cpu().numpy()

    def graphs(self, qp, lp, bufs, use_graph=True):
        """One callable per KV copy that runs the step: a captured graph's replay, or the kernel-by-kernel launches."""
        if not use_graph:
            return [(lambda c=c: self.step(qp, lp, bufs, c)) for c in range(self.kv_copies)], []
        keep = []
        runs = []
        for c in range(self.kv_copies):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                self.step(qp, lp, bufs, c)
            keep.append(g)
            runs.append(g.replay)
        return runs, keep


def timed_steps(runs, steps: int, warmup: int, world: int, min_steps: int, min_seconds: float):
    """Warm-up, then rounds of exactly `steps` back-to-back steps, each round between barrier + synchronize and timed
    with one pair of CUDA events (max over ranks); then as many steps again with an event after every step for the
    per-step distribution.  `runs` are rotated (independent KV copies)."""
    n = len(runs)
    k = 0
    for _ in range(max(20, warmup)):
        runs[k % n]()
        k += 1
    barrier(world)
    round_ms = []
    while True:
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier(world)
        start.record()
        for _ in range(steps):
            runs[k % n]()
            k += 1
        end.record()
        barrier(world)
        round_ms.append(max_over_ranks(start.elapsed_time(end), world))
        if len(round_ms) * steps >= min_steps and sum(round_ms) >= min_seconds * 1e3:
            break
        if len(round_ms) >= 4000:
            break
    total = len(round_ms) * steps
    m = min(total, 2000)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(m + 1)]
    ev[0].record()
    for j in range(m):
        runs[k % n]()
        k += 1
        ev[j + 1].record()
    torch.cuda.synchronize()
    per_step = [ev[j].elapsed_time(ev[j + 1]) for j in range(m)]
    return sum(round_ms) / total, round_ms, per_step


def profile_dense_cost(w: Workload, args, points: int, reps: int):
    """Step latency against the packed length: for every grid point the selector is forced to that length (a
    one-bucket table), the step is captured the way the arms run it and its replays are timed; the point is their median."""
    from paper_2607_14647_b200 import profiler
    cfg = w.cfg
    grid = cost_grid(cfg, points, w.is_layer)
    med, p25 = [], []
    for T in grid:
        w.ctx.set_cost_buckets(cfg.B, cfg.gamma, [T], [1.0])
        d = w.depths_now()
        qp, lp = w.pack(d)
        bufs = w.make_bufs(T)
        w.step(qp, lp, bufs)
        runs, keep = w.graphs(qp, lp, bufs, not args.no_graph)
        for r in runs[1:]:
            r()
        k = [0]

        def run():
            runs[k[0] % len(runs)]()
            k[0] += 1
        ts = profiler.time_replays(run, reps, 3, COST_INNER)
        med.append(float(np.median(ts)))
        p25.append(float(np.percentile(ts, 25)))
        del qp, lp, bufs, runs, keep
    if w.is_layer:     # cost moves in steps of the GEMM row blocks: keep the steps
        table = monotone_cost(np.interp(np.arange(cfg.t_cap + 1), grid, med))
    else:
        table = profiler.dense_table(grid, med, cfg.t_cap + 1)
    return grid, med, p25, table


def profile_bucket_cost(w: Workload, args, reps: int):
    """C(B, rho) for this workload's batch size at the paper's four ratio buckets: Appendix C's protocol through the
    library's cost grid (one captured batch size here; the bench has one)."""
    from paper_2607_14647_b200 import binding, profiler
    cfg = w.cfg
    grid = binding.CostGrid([cfg.B], RATIO_BUCKETS, cfg.gamma)

    def make_step(B, K):
        w.ctx.set_cost_buckets(cfg.B, cfg.gamma, [K], [1.0])
        d = w.depths_now()
        qp, lp = w.pack(d)
        bufs = w.make_bufs(K)
        w.step(qp, lp, bufs)
        runs, keep = w.graphs(qp, lp, bufs, not args.no_graph)
        k = [0]

        def run():
            runs[k[0] % len(runs)]()
            k[0] += 1
        run._keep = (qp, lp, bufs, keep)
        return run
    table = profiler.profile_cost_grid(grid, make_step, reps=reps, warmup=3, inner=COST_INNER)
    return grid, table


def run_arms(w: Workload, args, world: int, arms: dict, light: bool):
    """Times every arm; `arms` maps a name to a function that installs its cost table on the context."""
    cfg = w.cfg
    res = {}
    steps = args.steps
    min_steps = args.min_timed_steps if not light else max(40, args.min_timed_steps // 2)
    min_seconds = args.min_timed_seconds if not light else args.min_timed_seconds / 2
    for name, install in arms.items():
        install()
        d = w.depths_now()
        qp, lp = w.pack(d)
        T = int(d.sum()) + cfg.B
        bufs = w.make_bufs(T)
        w.step(qp, lp, bufs)
        # (a) kernel-by-kernel launches, with events around the verification forward (the roofline's kernel time)
        n_ev = max(steps, 40 if light else 100)
        for c in range(w.kv_copies):
            w.step(qp, lp, bufs, c)
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(n_ev)]
        barrier(world)
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        for k in range(n_ev):
            ev[k][0].record()
            so = w.select()
            ev[k][1].record()
            w.middle(qp, so, bufs, k % w.kv_copies)
            ev[k][2].record()
            w.accept(lp, so, bufs)
            ev[k][3].record()
        end.record()
        barrier(world)
        eager_ms = max_over_ranks(start.elapsed_time(end), world) / n_ev
        mid = [e[1].elapsed_time(e[2]) for e in ev]
        sel_ms = statistics.median(e[0].elapsed_time(e[1]) for e in ev)
        acc_ms = statistics.median(e[2].elapsed_time(e[3]) for e in ev)
        # (b) the same step captured once per KV copy in a CUDA graph and replayed: the packed length is read on the
        # device, so one graph serves whatever depth vector the selector produces
        runs, keep = w.graphs(qp, lp, bufs, not args.no_graph)
        mean_ms, round_ms, per_step = timed_steps(runs, steps, args.warmup, world, min_steps, min_seconds)
        accepted = int(bufs["total"].item())
        assert w.ctx.poll_device_status() == 0
        res[name] = dict(T=T, accepted=accepted, ms_per_step=mean_ms, per_step=stats_ms(per_step), rounds=len(round_ms),
                         timed_steps=len(round_ms) * steps, eager_ms=eager_ms, mid_ms=statistics.mean(mid), mid=stats_ms(mid),
                         tokens_per_s=world * accepted / (mean_ms * 1e-3), sel_ms=sel_ms, acc_ms=acc_ms,
                         attn_bytes=attn_algorithmic_bytes(cfg, w.sel.ctx_lens, d), depths=d)
        del qp, lp, bufs, runs, keep
    return res


def arms_json(w: Workload, res: dict, pk: dict) -> dict:
    out = {}
    for k, v in res.items():
        e = {"T": v["T"], "accepted_tokens": v["accepted"], "ms_per_step": round(v["ms_per_step"], 4),
             "ms_per_step_median": v["per_step"]["median"], "ms_per_step_p95": v["per_step"]["p95"],
             "timed_steps": v["timed_steps"], "ms_per_step_kernel_by_kernel": round(v["eager_ms"], 4),
             "tokens_per_s": round(v["tokens_per_s"], 1), "select_us_median": round(v["sel_ms"] * 1e3, 1),
             "accept_us_median": round(v["acc_ms"] * 1e3, 1),
             "accept_gbs": round(v["T"] * w.cfg.vocab * 2 / (v["acc_ms"] * 1e-3) / 1e9, 1)}
        if w.is_layer:
            e["forward_ms"] = round(v["mid_ms"], 4)
            e["forward_ms_median"] = v["mid"]["median"]
        else:
            gbs = v["attn_bytes"] / (v["mid_ms"] * 1e-3) / 1e9
            e.update({"attn_ms": round(v["mid_ms"], 4), "attn_ms_median": v["mid"]["median"], "attn_ms_p95": v["mid"]["p95"],
                      "attn_gbs": round(gbs, 1), "attn_frac_of_measured": round(gbs / pk["hbm_gbs"], 4),
                      "attn_frac_of_8000_nominal": round(gbs / 8000.0, 4)})
        out[k] = e
    return out


def standard_arms(w: Workload, cost_table, bucket_grid=None) -> dict:
    cfg = w.cfg
    cap = cfg.t_cap
    arms = {"pruned": lambda: w.ctx.set_cost_dense(cost_table),
            "full_gamma": lambda: w.ctx.set_cost_dense(np.ones(cap + 1, np.float32)),
            "gamma0": lambda: w.ctx.set_cost_dense((1.0 + 10.0 * np.maximum(0, np.arange(cap + 1) - cfg.B)).astype(np.float32))}
    if bucket_grid is not None:
        arms["paper_buckets"] = lambda: w.ctx.set_cost_from_grid(bucket_grid, cfg.B)
    return arms


def gemm_alone(w: Workload, res: dict, pk: dict, with_lm_head: bool):
    """The four projections of the layer, timed alone (tensor roofline), and the LM head fused with acceptance."""
    from paper_2607_14647_b200 import binding
    cfg, dev, ctx, cap = w.cfg, w.dev, w.ctx, w.cap
    gemm = {}
    qkv_w, q_w = (cfg.n_q_heads + 2 * cfg.n_kv_heads) * cfg.head_dim, cfg.n_q_heads * cfg.head_dim
    for arm in ("pruned", "full_gamma"):
        T = res[arm]["T"]
        cu1 = torch.tensor([0, T], dtype=torch.int32, device=dev)
        rows = {}
        for name, (wt, w2, mode, K, N) in {"qkv": (w.d_w["w_qkv"], None, 0, cfg.hidden, qkv_w),
                                           "o": (w.d_w["w_o"], None, 1, q_w, cfg.hidden),
                                           "gate_up_swiglu": (w.d_w["w_gate"], w.d_w["w_up"], 2, cfg.hidden, cfg.intermediate),
                                           "down": (w.d_w["w_down"], None, 1, cfg.intermediate, cfg.hidden)}.items():
            a_in = torch.randn((cap, K), device=dev, dtype=torch.float32).to(torch.bfloat16)
            outb = torch.empty((cap, N), dtype=torch.bfloat16, device=dev)
            resb = torch.zeros((cap, N), dtype=torch.bfloat16, device=dev) if mode == 1 else None
            for _ in range(3):
                ctx.gemm_bf16(a_in, wt, cu1, cap, outb, mode=mode, w2=w2, residual=resb)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(20):
                ctx.gemm_bf16(a_in, wt, cu1, cap, outb, mode=mode, w2=w2, residual=resb)
            e1.record()
            e1.synchronize()
            ms = e0.elapsed_time(e1) / 20
            fl = 2.0 * T * K * N * (2 if mode == 2 else 1)
            rows[name] = {"ms": round(ms, 4), "tflops": round(fl / ms / 1e9, 1), "frac_of_measured_burst": round(fl / ms / 1e9 / pk["bf16_tflops"], 4)}
        tot_ms = sum(r["ms"] for r in rows.values())
        tf = layer_flops(cfg, T) / tot_ms / 1e9
        rows["all"] = {"T": T, "ms": round(tot_ms, 4), "tflops": round(tf, 1), "frac_of_measured_burst": round(tf / pk["bf16_tflops"], 4)}
        gemm[arm] = rows
    if with_lm_head:
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

            fused_ms = timed(lambda: ctx.lm_head_accept(xh, w_lm[:V], w.d_draft, cu_full, cap, out_tokens=False))
            gemm_ms = timed(lambda: ctx.gemm_bf16(xh, w_lm, cu_full, cap, logits_buf))
            ctx_v = binding.Context(max_B=cfg.B, max_gamma=cfg.gamma, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
                                    head_dim=cfg.head_dim, page_size=cfg.page_size, max_pages_per_req=1, vocab=Vp)
            acc_ms = timed(lambda: ctx_v.accept(logits_buf, w.d_draft, cu_full, cap, out_tokens=False))
            fl = 2.0 * T * cfg.hidden * V
            gemm["lm_head"] = {"T": T, "V": V, "fused_ms": round(fused_ms, 4), "fused_tflops": round(fl / fused_ms / 1e9, 1),
                               "frac_of_measured_burst": round(fl / fused_ms / 1e9 / pk["bf16_tflops"], 4),
                               "unfused_gemm_ms": round(gemm_ms, 4), "unfused_accept_ms": round(acc_ms, 4),
                               "logits_bytes_not_moved": 2 * T * V * 2}
            ctx_v.close()
            del w_lm, logits_buf, ctx_v
        except Exception as exc:   # the extra measurement must not take the bench line down
            gemm["lm_head"] = {"error": repr(exc)[:200]}
    return gemm


def stochastic_extra(w: Workload, cost):
    """Stochastic variant (causal selector + rejection-sampling acceptance), timed alone at full depth."""
    cfg, dev, ctx, cap = w.cfg, w.dev, w.ctx, w.cap
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
        so = w.sel_out
        t_sel = timed_us(lambda: ctx.select(w.d_conf, w.d_draft, w.d_bonus, w.d_ctx, out=so))
        t_selc = timed_us(lambda: ctx.select(w.d_conf, w.d_draft, w.d_bonus, w.d_ctx, out=so, causal=True))
        ctx.enable_plan_in_select(False)
        t_sel_np = timed_us(lambda: ctx.select(w.d_conf, w.d_draft, w.d_bonus, w.d_ctx, out=so))
        ctx.enable_plan_in_select(True)
        full = np.full(cfg.B, cfg.gamma, np.int32)
        cu_full = torch.from_numpy(wl.cu_q_from_depths(full)).to(dev)
        # drafter logits: the target rows plus noise (generated on the device; the values do not change the traffic)
        idx = torch.from_numpy(np.concatenate([i * (cfg.gamma + 1) + np.arange(cfg.gamma) for i in range(cfg.B)])).to(dev)
        d_dl = w.d_logits_all.index_select(0, idx).view(cfg.B, cfg.gamma, cfg.vocab).contiguous()
        d_dl += (0.3 * torch.randn(d_dl.shape, device=dev, dtype=torch.float32)).to(torch.bfloat16)
        ua_np, us_np = wl.uniforms(cfg)
        d_ua, d_us = torch.from_numpy(ua_np).to(dev), torch.from_numpy(us_np).to(dev)
        dr = (w.d_draft % cfg.vocab).contiguous()
        t_rs = timed_us(lambda: ctx.accept_rs(w.d_logits_all, d_dl, dr, cu_full, cap, d_ua, d_us), n=10)
        rs_bytes = 2 * cfg.vocab * (cfg.t_cap + cfg.B * cfg.gamma)
        out = {"select_us": round(t_sel, 2), "select_without_attention_work_list_us": round(t_sel_np, 2),
               "select_causal_us": round(t_selc, 2), "accept_rs_us": round(t_rs, 1), "accept_rs_scan_bytes": rs_bytes,
               "accept_rs_gbs": round(rs_bytes / (t_rs * 1e-6) / 1e9, 1)}
        del d_dl
        return out
    except Exception as exc:   # the extra measurement must not take the bench line down
        return {"error": repr(exc)[:200]}


def e2e_hidden_form(w: "Workload", args, cost, h: dict, want_accepted: int, hidden: int = 4096):
    """The end-to-end step again, in the host call's hidden-state form: the kept rows of the last hidden states
    (8 KB each) cross the bus instead of the kept logits rows (300 KB each), and the step ends in the LM head fused
    with acceptance (the LM head's weights are resident like the cache).  A longer step (it contains the LM-head GEMM)
    that is no longer bound by the bus."""
    from paper_2607_14647_b200 import binding
    cfg, dev = w.cfg, w.dev
    ctx = binding.Context(max_B=cfg.B, max_gamma=cfg.gamma, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
                          head_dim=cfg.head_dim, page_size=cfg.page_size, max_pages_per_req=w.kv.block_table.shape[1],
                          vocab=cfg.vocab, hidden=hidden, intermediate=hidden)
    try:
        ctx.set_cost_dense(cost)
        w_lm = wl.lm_head_weight(cfg, vocab=cfg.vocab, hidden=hidden)
        full = np.full(cfg.B, cfg.gamma, np.int32)
        x_all = wl.lm_head_x_rows(cfg, w.sel, full, w_lm).view(cfg.B, cfg.gamma + 1, hidden).contiguous().pin_memory()
        d_w = w_lm.to(dev)
        hout = ctx.host_step_outputs(cfg.B, cfg.gamma)
        call = lambda: ctx.verify_step_host(h["conf"], h["draft"], h["bonus"], h["ctx"], h["bt"], h["q"], None, w.d_k[0], w.d_v[0],
                                            out=hout, hidden_rows=x_all, w_lm=d_w)
        for _ in range(3):
            call()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            call()
        torch.cuda.synchronize()
        dt = (time.perf_counter() - t0) / args.e2e_steps
        acc = int(hout["n_accepted_total"].item())
        assert ctx.poll_device_status() == 0
        return {"value": acc / dt, "unit": UNIT, "ms_per_step": round(dt * 1e3, 4), "accepted_tokens": acc,
                "accepted_tokens_of_the_logits_form": want_accepted, "h2d_bytes_per_step": hout["h2d_bytes"],
                "d2h_bytes_per_step": hout["d2h_bytes"], "hidden": hidden,
                "api": "dcut_verify_step_host with hidden_rows + w_lm (select, attention, LM head fused with acceptance)"}
    finally:
        ctx.close()


def multistep_arm(cfg, dev, args, world, cost, n_chain: int):
    """`n_chain` consecutive verify steps chained on the device in one graph: select -> attention -> accept -> commit,
    the commit advancing every request's context by its accepted drafts + 1 and handing its bonus token to the next
    step; nothing returns to the host in between.  (No drafter here: every step reads the same confidences and the
    same packed query / logits rows; the contexts, and with them the KV each step streams, grow from step to step.)"""
    spare = 2 + (n_chain * (cfg.gamma + 1) + cfg.page_size - 1) // cfg.page_size
    w = Workload(cfg, dev, kv_copies=1, spare_pages=spare)
    try:
        # block table with room for the chain's growth: the extra columns point at the spare pages (read-only here)
        used = set(w.kv.block_table[w.kv.block_table >= 0].tolist())
        spare_ids = [pid for pid in range(w.kv.num_pages) if pid not in used][:spare]
        assert len(spare_ids) == spare
        ext = torch.tensor(spare_ids, dtype=torch.int32, device=dev).repeat(cfg.B, 1)
        pages = ((w.sel.ctx_lens.astype(np.int64) + cfg.gamma + 1 + cfg.page_size - 1) // cfg.page_size)
        width = int(pages.max()) + spare
        bt = torch.full((cfg.B, width), -1, dtype=torch.int32, device=dev)
        bt[:, : w.d_bt.shape[1]] = w.d_bt
        for i in range(cfg.B):
            bt[i, int(pages[i]): int(pages[i]) + spare] = ext[i]
        w.close()
        from paper_2607_14647_b200 import binding
        w.ctx = binding.Context(max_B=cfg.B, max_gamma=cfg.gamma, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
                                head_dim=cfg.head_dim, page_size=cfg.page_size, max_pages_per_req=width, vocab=cfg.vocab)
        w.ctx.enable_plan_in_select(True)
        w.d_bt = bt
        w.ctx.set_cost_dense(cost)
        d = w.depths_now()
        qp, lp = w.pack(d)
        T = int(d.sum()) + cfg.B
        bufs = w.make_bufs(T)
        ctx0, bonus0 = w.d_ctx.clone(), w.d_bonus.clone()
        max_ctx = width * cfg.page_size
        acc_sum = torch.zeros(1, dtype=torch.int32, device=dev)

        def chain():
            w.d_ctx.copy_(ctx0)
            w.d_bonus.copy_(bonus0)
            acc_sum.zero_()
            for _ in range(n_chain):
                w.step(qp, lp, bufs)
                w.ctx.commit(bufs["accept_len"], bufs["out_tokens"], w.d_ctx, w.d_bonus, max_ctx)
                acc_sum.add_(bufs["total"])

        chain()
        torch.cuda.synchronize()
        assert w.ctx.poll_device_status() == 0
        if args.no_graph:
            runs = [chain]
            keep = []
        else:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                chain()
            runs, keep = [g.replay], [g]
        mean_ms, round_ms, per = timed_steps(runs, max(4, args.steps // n_chain), args.warmup // 2, world,
                                             max(10, args.min_timed_steps // n_chain), args.min_timed_seconds / 2)
        accepted = int(acc_sum.item())
        assert w.ctx.poll_device_status() == 0
        grown = int((w.d_ctx - ctx0).sum().item())
        return {"steps_chained": n_chain, "ms_per_chain": round(mean_ms, 4), "ms_per_step": round(mean_ms / n_chain, 4),
                "ms_per_chain_median": stats_ms(per)["median"], "accepted_tokens_per_chain": accepted,
                "context_tokens_committed": grown, "tokens_per_s": round(world * accepted / (mean_ms * 1e-3), 1),
                "launches_per_step": 6, "note": "select -> verify_attn -> accept -> commit, all on the device, one graph for the chain"}
    finally:
        w.close()


def bench_workload(cfg, dev, args, world, rank, local, headline: bool):
    """All measurements of one workload; returns the section that goes on the JSON line."""
    pk = peaks()
    light = not headline
    w = Workload(cfg, dev)
    try:
        points = args.cost_points if headline else max(8, args.cost_points // 2)
        reps = args.cost_reps if headline else max(7, args.cost_reps // 2)
        grid, med, p25, cost = profile_dense_cost(w, args, points, reps)
        bucket_grid, bucket_table = profile_bucket_cost(w, args, reps)
        sampler = ClockSampler(local) if rank == 0 else None
        res = run_arms(w, args, world, standard_arms(w, cost, bucket_grid), light)
        clocks = sampler.stop() if sampler else {}
        section = {"workload": workload_name(cfg), "arms": arms_json(w, res, pk), "clocks": clocks,
                   "l2": (f"{w.kv_copies} independent copies of the KV cache are rotated step by step "
                          f"({2 * w.kv.k_cache.numel() * 2 / 1e6:.0f} MB each; L2 is 126 MB)" if w.kv_copies > 1 else
                          f"inputs exceed L2: each step streams {res['pruned']['attn_bytes'] / 1e6:.0f} MB of KV and "
                          f"{res['pruned']['T'] * cfg.vocab * 2 / 1e6:.0f} MB of logits once (L2 is 126 MB)"),
                   "cost_table": {"points_T": grid, "median_ms": [round(x, 4) for x in med], "p25_ms": [round(x, 4) for x in p25],
                                  "table_ms_at_points": [round(float(cost[t]), 4) for t in grid],
                                  "fit": "running minimum from the long end" if w.is_layer else "isotonic (non-decreasing least squares)",
                                  "reps_per_point": reps, "steps_per_rep": COST_INNER},
                   "bucket_cost_table": {"B": cfg.B, "ratios": [f"{n}/{d}" for n, d in RATIO_BUCKETS],
                                         "K": [bucket_grid.budget(cfg.B, r) for r in range(len(RATIO_BUCKETS))],
                                         "median_ms": [round(float(x), 4) for x in bucket_table[0]]}}
        if w.is_layer and rank == 0:
            section["gemm_alone"] = gemm_alone(w, res, pk, with_lm_head=True)
            section["flops_per_token"] = layer_flops(cfg, 1)
        return section, res, cost, w
    except Exception:
        w.close()
        raise


def run_attn_only(args):
    """dcut_verify_attn alone, a few launches per arm: the command the ncu captures under profiles/ run."""
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    cfg = wl.config(args.config)
    if args.batch > 0:
        cfg = dataclasses.replace(cfg, B=args.batch, name=f"{cfg.name}_B{args.batch}")
    w = Workload(cfg, dev, kv_copies=1)
    cost = wl.cost_table_linear(cfg.t_cap + 1, 0.2, 0.0001)
    out = {}
    for name, install in standard_arms(w, cost).items():
        install()
        d = w.depths_now()
        qp, _ = w.pack(d)
        bufs = w.make_bufs(int(d.sum()) + cfg.B)
        so = w.select()
        for _ in range(args.warmup):
            w.middle(qp, so, bufs)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for a, b in ev:
            a.record()
            w.middle(qp, so, bufs)
            b.record()
        torch.cuda.synchronize()
        by = attn_algorithmic_bytes(cfg, w.sel.ctx_lens, d)
        ms = statistics.median(a.elapsed_time(b) for a, b in ev)
        out[name] = {"T": int(d.sum()) + cfg.B, "algorithmic_bytes": by, "attn_ms_median": round(ms, 4), "attn_gbs": round(by / ms / 1e6, 1)}
    assert w.ctx.poll_device_status() == 0
    w.close()
    print(json.dumps({"attn_only": workload_name(cfg), "arms": out}))


def run_dcut(args):
    world, rank, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    pk = peaks()
    cfg = wl.config(args.config)
    if args.gamma > 0:
        cfg = dataclasses.replace(cfg, gamma=args.gamma, name=f"{cfg.name}_gamma{args.gamma}")
    section, res, cost, w = bench_workload(cfg, dev, args, world, rank, local, headline=True)
    is_layer = w.is_layer
    sel, kv = w.sel, w.kv

    # what the stored profile (the table --impl reference reads: that arm has no GPU) would have selected
    stored = stored_cost_profile(cfg)
    stored_T = None
    if stored is not None and not is_layer:
        from paper_2607_14647_b200 import profiler
        w.ctx.set_cost_dense(profiler.dense_table(stored["T"], stored["median_ms"], cfg.t_cap + 1))
        stored_T = int(w.depths_now().sum()) + cfg.B
    q_all_host, logits_all_host = w.q_all_host, w.logits_all_host

    # ---- end to end from host buffers ---------------------------------------------------------
    e2e = None
    try:
        w.ctx.set_cost_dense(cost)
        if not is_layer and args.e2e_steps > 0:
            pin = lambda t: t.contiguous().pin_memory()
            h = dict(conf=pin(torch.from_numpy(sel.conf)), draft=pin(torch.from_numpy(sel.draft_ids)),
                     bonus=pin(torch.from_numpy(sel.bonus_ids)), ctx=pin(torch.from_numpy(sel.ctx_lens)),
                     bt=pin(torch.from_numpy(kv.block_table)), q=pin(w.q_all_host), logits=pin(w.logits_all_host))
            hout = w.ctx.host_step_outputs(cfg.B, cfg.gamma)
            call = lambda: w.ctx.verify_step_host(h["conf"], h["draft"], h["bonus"], h["ctx"], h["bt"], h["q"], h["logits"],
                                                  w.d_k[0], w.d_v[0], out=hout)
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
        stochastic = stochastic_extra(w, cost) if (not is_layer and rank == 0) else None
        e2e_hidden = None
        if not is_layer and world == 1 and args.e2e_steps > 0:
            try:
                e2e_hidden = e2e_hidden_form(w, args, cost, h, res["pruned"]["accepted"])
            except Exception as exc:   # the extra measurement must not take the bench line down
                e2e_hidden = {"error": repr(exc)[:300]}
    finally:
        w.close()
    del w
    torch.cuda.empty_cache()

    multistep = None
    if args.multistep > 0 and not is_layer:
        try:
            multistep = multistep_arm(cfg, dev, args, world, cost, args.multistep)
        except Exception as exc:
            multistep = {"error": repr(exc)[:300]}
        torch.cuda.empty_cache()

    # ---- bounded runs of the other workloads (one GPU only) -----------------------------------------
    extras = {}
    want = []
    if args.extras == "auto":
        want = [1, 3, 4] if (world == 1 and args.config == 2 and args.gamma == 0) else []
    elif args.extras != "none":
        want = [int(x) for x in args.extras.split(",") if x.strip()]
    for idx in want:
        if idx == cfg.index:
            continue
        try:
            t0 = time.perf_counter()
            sec, r2, _, w2 = bench_workload(wl.config(idx), dev, args, world, rank, local, headline=False)
            w2.close()
            del w2
            sec["bench_seconds"] = round(time.perf_counter() - t0, 1)
            extras[str(idx)] = sec
        except Exception as exc:   # an extra must not take the headline down
            extras[str(idx)] = {"error": repr(exc)[:300]}
        torch.cuda.empty_cache()

    if rank != 0:
        return
    p = res["pruned"]
    if args.write_cost_profile:
        os.makedirs(COST_PROFILE_DIR, exist_ok=True)
        ct = section["cost_table"]
        json.dump({"B": cfg.B, "gamma": cfg.gamma, "workload": workload_name(cfg), "T": ct["points_T"], "median_ms": ct["median_ms"],
                   "protocol": "bench.py profile_dense_cost: selector forced to T, the step's CUDA graph replayed, median of "
                               f"{ct['reps_per_point']} samples of {ct['steps_per_rep']} back-to-back replays per point", "gpu": torch.cuda.get_device_name(local)},
                  open(os.path.join(COST_PROFILE_DIR, f"b200_config{cfg.index}_gamma{cfg.gamma}.json"), "w"), indent=1)
    line = {
        "metric": METRIC, "value": p["tokens_per_s"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(20, args.warmup), "ms_per_step": p["ms_per_step"], "ms_per_step_median": p["per_step"]["median"],
        "ms_per_step_p95": p["per_step"]["p95"], "timed_steps": p["timed_steps"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload_name(cfg), "arm": "D-cut pruned", "cost_table": COST_TABLE_NOTE,
                   "launch": "kernel by kernel" if args.no_graph else "one CUDA graph of the step, replayed each step",
                   "timing": f"rounds of {args.steps} back-to-back replays until >= {args.min_timed_steps} steps and >= "
                             f"{args.min_timed_seconds} s; mean over all; median / p95 from individually timed replays",
                   "l2": section["l2"], "parallelism": "replicas only" if world > 1 else "1 GPU"},
        "cost_table_source": "profiled live on this GPU",
        "arms": section["arms"],
        "e2e": e2e,
        "gpu_launches": (13 if is_layer else 5) * args.steps,
        "cost_table_ms": section["cost_table"], "bucket_cost_table": section["bucket_cost_table"],
        "clocks": section["clocks"],
    }
    if stored_T is not None:
        line["cost_table_stored_profile"] = {"T_it_selects": stored_T, "T_live_profile_selects": p["T"],
                                             "note": "the stored profile is what --impl reference reads (no GPU on that arm)"}
    if not is_layer:
        achieved = p["attn_bytes"] / (p["mid_ms"] * 1e-3) / 1e9
        line["roofline"] = {"kernel": "dcut_verify_attn (attn_item_kernel + attn_combine_kernel; the work list is built in dcut_select_kernel)",
                            "bound": "hbm", "achieved": round(achieved, 1), "peak": pk["hbm_gbs"], "unit": "GB/s",
                            "frac": round(achieved / pk["hbm_gbs"], 4), "peak_source": f"of {pk['source']}",
                            "frac_of_8000_nominal": round(achieved / 8000.0, 4),
                            "algorithmic_bytes_per_launch": p["attn_bytes"], "launch_ms_mean": round(p["mid_ms"], 4),
                            "launch_ms_median": p["mid"]["median"], "launches_timed": p["mid"]["n"],
                            "traffic": int(ATTN_TRAFFIC_RATIO * p["attn_bytes"]),
                            "traffic_source": "ncu dram bytes per algorithmic byte on this workload's shapes (profiles/attn_item_kernel_dram_traffic.md) x this launch's algorithmic bytes"}
    else:
        g = section["gemm_alone"]["full_gamma"]["all"]
        line["config"]["arm"] += "; verification forward = one decoder layer (dcut_layer_forward)"
        line["layer"] = {"gemm_alone": section["gemm_alone"], "flops_per_token": section["flops_per_token"]}
        line["roofline"] = line["roofline_tensor"] = {
            "kernel": "gemm_tcgen05_kernel (4 projections of the layer, full-gamma arm, timed alone)", "bound": "tensor",
            "achieved": g["tflops"], "peak": pk["bf16_tflops"], "unit": "TFLOP/s", "frac": round(g["tflops"] / pk["bf16_tflops"], 4),
            "peak_source": f"of {pk['source']} (burst)", "traffic": None}
    if e2e_hidden is not None:
        line["e2e_hidden_state_form"] = e2e_hidden
    if stochastic is not None:
        line["stochastic"] = stochastic
    if multistep is not None:
        line["multistep"] = multistep
    if extras:
        line["configs"] = extras
    if world == 1 and not args.no_cpu_baseline and not is_layer:
        info, *_ = oracle_sample(cfg, sel, kv, q_all_host, logits_all_host, cost, args.cpu_seconds)
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
    ctx.enable_plan_in_select(True)
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
        for _ in range(max(3, min(args.warmup, 5))):
            step()
        eager_ms, fwd_ms = timed(min(args.steps, 20))
        ms, per = eager_ms, None
        if not args.no_graph:
            # the same step captured once in a CUDA graph and replayed (the packed length is read on the device)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            ms, _, per_step = timed_steps([graph.replay], min(args.steps, 20), 5, world, 40, 0.5)
            per = stats_ms(per_step)
            del graph
        assert ctx.poll_device_status() == 0
        planted = int((np.minimum(d, sel.reject_index) + 1).sum())
        res[name] = {"T": T, "ms_per_step": round(ms, 4), "ms_per_step_median": per["median"] if per else None,
                     "ms_per_step_p95": per["p95"] if per else None,
                     "ms_per_step_kernel_by_kernel": round(eager_ms, 4), "forward_ms": round(fwd_ms, 4),
                     "accepted_tokens_planted": planted, "accepted_tokens_by_the_random_init_model": int(state["out"][3].item()),
                     "tokens_per_s": round(world * planted / (ms * 1e-3), 1),
                     "verified_tokens_per_s": round(world * T / (ms * 1e-3), 1),
                     "forward_tflops": round(flops_tok * T / fwd_ms / 1e9, 1),
                     "kv_streamed_gb": round(L * attn_algorithmic_bytes(cfg, sel.ctx_lens, d) / 1e9, 2)}
    clocks = sampler.stop() if sampler else {}
    if rank != 0:
        return
    pkj = peaks()
    tf_peak = pkj["bf16_tflops_sustained"]
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
                     "peak_source": f"of {pkj['source']} (sustained)", "traffic": None},
        "e2e": None, "gpu_launches": (5 + 10 * L) * args.steps,   # select (with the attention work list), embed, 10 per layer, norm, LM head, match
        "cost_table_ms": {str(t): round(c, 4) for t, c in zip(grid, prof)}, "clocks": clocks,
    }
    print(json.dumps(line))


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.attn_only:
        run_attn_only(args)
    elif args.layers > 0:
        run_model(args)
    else:
        run_dcut(args)


if __name__ == "__main__":
    main()
