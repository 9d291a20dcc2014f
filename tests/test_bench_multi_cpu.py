"""The N > 1 plumbing of bench.py on CPU: two `gloo` ranks exercise the max-over-ranks timing and
the whole-job aggregation, and the reference arm under a 2-rank launch prints exactly one line
(rank 0) while the other rank exits 0 without work.  The data path itself has no collective: ranks
are independent replicas."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
alone = bench.max_over_ranks(3.0, None, torch.device("cpu"))
val = bench.whole_job_value(world, 1000, ms)
dist.barrier()
dist.destroy_process_group()
print(json.dumps({{"rank": rank, "ms": ms, "alone": alone, "value": val}}), flush=True)
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _launch(world, argv):
    port = _free_port()
    procs = []
    for r in range(world):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable] + argv, env=env, cwd=ROOT, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=300)
        assert p.returncode == 0, e[-2000:]
        outs.append(o)
    return outs


def test_max_over_ranks_and_aggregate_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER.format(root=ROOT))
    outs = _launch(2, [str(script)])
    rows = sorted((json.loads(o.strip().splitlines()[-1]) for o in outs), key=lambda r: r["rank"])
    assert [r["rank"] for r in rows] == [0, 1]
    for r in rows:
        assert r["ms"] == 15.0            # the slower rank's time, on every rank
        assert r["alone"] == 3.0
        assert r["value"] == 2 * 1000 / 15e-3


def test_reference_arm_two_ranks_prints_one_line():
    outs = _launch(2, ["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                       "--workload", "tiny"])
    lines = [l for o in outs for l in o.splitlines() if l.strip()]
    assert len(lines) == 1 and outs[1].strip() == ""
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["config"]["workload"] == "tiny"
