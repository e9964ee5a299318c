"""Host-side logic of the N > 1 benchmark path, run as two gloo ranks on the CPU:
the max-over-ranks reduction that turns per-rank times into the reported time, and
the rule that only rank 0 of the reference arm prints."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["ECQ_ROOT"])
import torch.distributed as dist
import bench
rank, local, world = bench.dist_env()
dist.init_process_group("gloo", rank=rank, world_size=world)
vals = [10.0 + rank, 5.0 - rank, 7.0]
out = bench.max_over_ranks(vals, world)
dist.barrier()
print(json.dumps({"rank": rank, "world": world, "out": out}))
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _env(rank, world, port):
    env = dict(os.environ)
    env.update({"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world),
                "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port), "ECQ_ROOT": ROOT})
    return env


def test_max_over_ranks_two_gloo_ranks():
    port = _free_port()
    procs = [subprocess.Popen([sys.executable, "-c", WORKER], env=_env(r, 2, port),
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True)
             for r in range(2)]
    outs = [p.communicate(timeout=180) for p in procs]
    for p, (so, se) in zip(procs, outs):
        assert p.returncode == 0, se[-2000:]
    for so, _ in outs:
        res = json.loads(so.strip().splitlines()[-1])
        assert res["world"] == 2 and res["out"] == [11.0, 5.0, 7.0]


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], 1) == [1.5, 2.5]


def test_reference_arm_prints_on_rank0_only():
    args = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
            "--steps", "1", "--warmup", "0", "--workload", "gauss_1m", "--ref-elems", "65536"]
    r1 = subprocess.run(args, env=_env(1, 2, _free_port()), capture_output=True, text=True, timeout=300)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = subprocess.run(args, env=_env(0, 2, _free_port()), capture_output=True, text=True, timeout=300)
    assert r0.returncode == 0, r0.stderr[-2000:]
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["metric"] == "codec_step_throughput" and line["unit"] == "GB/s"


def test_step_bytes_closed_form():
    sys.path.insert(0, ROOT)
    import bench
    from paper_1806_08054_b200 import workloads as wl
    w = wl.WORKLOADS["resnet50"]
    enc, dec = bench.step_bytes(w)
    words = -(-w.d * 5 // 32)
    nb = -(-w.d // 512)
    assert enc == 12 * w.d + 4 * words + 4 * nb
    assert dec == 8 * (4 * words + 4 * nb) + 4 * w.d
