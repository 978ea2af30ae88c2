"""Host-side logic of bench.py: byte accounting, and the one cross-rank exchange of the N > 1
path (barrier + max over ranks), run as two gloo ranks on CPU."""
import os
import socket
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_RANK_SCRIPT = r"""
import os, sys
sys.path.insert(0, os.environ["DCUT_ROOT"])
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
bench.barrier(world)
slowest = bench.max_over_ranks(10.0 * (rank + 1), world)
assert slowest == 10.0 * world, slowest
# whole-job value: every rank processes the same units; the job is as slow as its slowest rank
units = 300
value = world * units / (slowest * 1e-3)
assert abs(value - world * units / (10.0 * world * 1e-3)) < 1e-9
bench.barrier(world)
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_max_over_ranks_with_two_gloo_ranks():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), DCUT_ROOT=ROOT, CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, "-c", _RANK_SCRIPT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for p in procs:
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0, out
        assert "ok" in out


def test_attention_byte_accounting():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2607_14647_b200 import workloads as wl
    cfg = wl.custom_config(B=2, gamma=4, n_q_heads=8, n_kv_heads=2, head_dim=128)
    ctx_lens = np.array([10, 33], np.int32)
    depths = np.array([0, 3], np.int32)
    # request 0: 11 cache tokens, 1 page, 1 query token; request 1: 37 tokens, 3 pages, 4 query tokens
    kv = (11 + 37) * 2 * 128 * 2 * 2
    qo = 2 * 5 * 8 * 128 * 2
    bt = (1 + 3) * 4 * 2
    assert bench.attn_algorithmic_bytes(cfg, ctx_lens, depths) == kv + qo + bt


def test_reference_arm_runs_without_gpu():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "0",
                          "--steps", "1", "--warmup", "0", "--cpu-seconds", "2"], capture_output=True, text=True,
                         timeout=300, env=dict(os.environ, CUDA_VISIBLE_DEVICES=""))
    assert out.returncode == 0, out.stderr
    import json
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0


def test_cost_grid_marks_the_row_block_steps():
    """Cost-table sample points: evenly spaced for the attention workloads; for the layer workloads the last length
    of a 128-row block and the first of the next, always with both ends."""
    sys.path.insert(0, ROOT)
    import bench
    from paper_2607_14647_b200 import workloads as wl
    cfg2, cfg4 = wl.config(2), wl.config(4)
    even = bench.cost_grid(cfg2, 18, False)
    assert even[0] == cfg2.B and even[-1] == cfg2.t_cap and len(even) == 18 and even == sorted(even)
    steps = np.diff(even)
    assert steps.max() - steps.min() <= 1
    tiled = bench.cost_grid(cfg4, 18, True)
    assert tiled[0] == cfg4.B and tiled[-1] == cfg4.t_cap and tiled == sorted(set(tiled))
    inner = tiled[1:-1]
    assert len(inner) % 2 == 0 and all(a % 128 == 0 and b == a + 1 for a, b in zip(inner[::2], inner[1::2]))
    assert [a for a in inner[::2]] == list(range(128, cfg4.t_cap, 128))          # every block edge at 18 points
    few = bench.cost_grid(cfg4, 6, True)
    assert few[0] == cfg4.B and few[-1] == cfg4.t_cap and 4 <= len(few) <= 8


def test_monotone_cost_ignores_a_disturbed_point():
    sys.path.insert(0, ROOT)
    import bench
    clean = np.array([1.0, 1.1, 1.2, 1.3, 1.4, 1.5], np.float32)
    noisy = clean.copy()
    noisy[2] = 1.9                                   # one measurement hit by interference
    out = bench.monotone_cost(noisy)
    assert (np.diff(out) >= 0).all()
    assert np.allclose(out, [1.0, 1.1, 1.3, 1.3, 1.4, 1.5])       # the spike is capped by the next clean point
    assert np.allclose(bench.monotone_cost(clean), clean)
