"""N > 1 runs replicas: one process per rank, no collective on the data path; only
the timing is reduced (maximum over ranks).  Checked here with two gloo ranks on CPU."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def test_two_ranks_reduce_time_by_max_and_sum_throughput(tmp_path):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()),
           os.path.join(ROOT, "tests", "gloo_worker.py"), str(tmp_path)]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    outs = [json.load(open(tmp_path / ("rank%d.json" % r))) for r in range(2)]
    for o in outs:
        assert o["world"] == 2
        assert o["ms"] == 15.0                         # the slowest rank sets the time
        assert abs(o["value"] - 2 * 100 / 15e-3) < 1e-6  # both replicas' ticks over that time
    assert outs[0]["seed"] != outs[1]["seed"]            # replicas draw different samples


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=120, env=env)
    assert res.returncode == 0 and res.stdout.strip() == ""
