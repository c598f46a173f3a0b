"""Multi-rank host logic of bench.py on CPU: world-size-2 gloo ranks aggregate like the GPU run does
(max over ranks of the step time, sum over ranks of the units), and the reference leg runs on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
import bench
rank = int(os.environ["RANK"])
dist.init_process_group("gloo", init_method="env://")
ms, units = bench.aggregate_over_ranks(1.0 + rank, 100.0 * (rank + 1), dist)
print(json.dumps({"rank": rank, "ms": ms, "units": units}))
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_aggregate_over_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err
        outs.append(json.loads(out.strip().splitlines()[-1]))
    for o in outs:
        assert o["ms"] == 2.0            # max over ranks
        assert o["units"] == 300.0       # sum over ranks


def test_aggregate_single_process():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.aggregate_over_ranks(3.5, 7.0, None) == (3.5, 7.0)
    assert bench.algorithmic_bytes(4, 2048, 5120, 80) == {"quantize_pack": 26460160, "dequant_reduce": 42926080}
    assert bench.payload_bytes(2048, 5120, 80) == 5488640


def test_reference_leg_runs_on_rank0_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
