"""Host-side logic of the benchmark that needs no GPU: the reference arm's JSON line, the clock-log
parser, and the rank layout of a 2-process run (gloo on CPU): every rank draws its own batch and rank 0
alone reports, with the max over ranks of the timing."""
import json
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c0",
                          "--steps", "1", "--warmup", "1"], capture_output=True, text=True, check=True).stdout.strip().splitlines()
    assert len(out) == 1
    d = json.loads(out[0])
    assert d["impl"] == "reference" and d["unit"] == "frames/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["vs_baseline"] is None


def test_per_rank_batches_differ_and_are_reproducible():
    import tw_synth
    cfg = tw_synth.get_config("c0")
    a, _ = tw_synth.make_encoder_batch(cfg.with_(seed=cfg.seed + 1000 * 0))
    b, _ = tw_synth.make_encoder_batch(cfg.with_(seed=cfg.seed + 1000 * 1))
    b2, _ = tw_synth.make_encoder_batch(cfg.with_(seed=cfg.seed + 1000 * 1))
    assert not np.array_equal(a, b) and np.array_equal(b, b2)


_WORKER = r"""
import os, sys, json
import torch, torch.distributed as dist
sys.path.insert(0, %r)
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
# the aggregation bench.py applies to its timings: max over ranks, frames summed over ranks
ms = torch.tensor([10.0 + 5.0 * rank], dtype=torch.float64)
dist.all_reduce(ms, op=dist.ReduceOp.MAX)
frames = 100
value = world * frames / (ms.item() * 1e-3)
dist.barrier()
if rank == 0:
    print(json.dumps({"ms": ms.item(), "value": value, "world": world}))
dist.destroy_process_group()
"""


def test_two_rank_timing_aggregation_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER % ROOT)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29613")
    res = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29613", str(script)],
                         capture_output=True, text=True, env=env, timeout=240)
    assert res.returncode == 0, res.stderr[-2000:]
    line = [l for l in res.stdout.splitlines() if l.startswith("{")][-1]
    d = json.loads(line)
    assert d["world"] == 2 and d["ms"] == 15.0 and abs(d["value"] - 2 * 100 / 0.015) < 1e-6


def test_clock_log_parser(tmp_path):
    import bench
    s = bench.ClockSampler.__new__(bench.ClockSampler)
    f = open(tmp_path / "c.csv", "w+")
    f.write("0, 1965, 1965, 700.1, 0x0, Not Active, Not Active, Not Active, Not Active\n"
            "0, 1350, 1965, 990.0, 0x4, Not Active, Not Active, Not Active, Active\n"
            "0, 1400, 1965, 990.0, 0x4, Not Active, Not Active, Not Active, Active\n")
    f.flush()

    class P:
        def terminate(self): pass
        def wait(self, timeout=None): pass
    s.f, s.p = f, P()
    out = s.stop()
    assert out["sm_mhz"] == 1400 and out["sm_max_mhz"] == 1965 and out["reasons"] == ["sw_power_cap"] and out["samples"] == 3
