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


def test_stage_split_plan_and_stamp_protocol_on_two_ranks(tmp_path):
    # stage split (Section 2.1: stages split over GPUs): both ranks get the same plan from the
    # library, the tick stamps keep them at most one tick apart, and a rank that leaves between
    # ticks is noticed on the host before the other one's next tick
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()),
           os.path.join(ROOT, "tests", "gloo_split_worker.py"), str(tmp_path)]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    outs = [json.load(open(tmp_path / ("split_rank%d.json" % r))) for r in range(2)]
    assert all(o["plans_equal"] for o in outs)
    plan = outs[0]["plan"]
    assert plan[0][0] == 0 and plan[0][1] == plan[1][0] and plan[1][1] == 6      # contiguous, all 6 stages
    # five 2048x2048 stages and a 2048x10 one: balanced by bytes puts three large stages on the first rank
    assert plan[0] == [0, 3]
    for o in outs:
        for e in o["log"]:
            assert e["ok"], (o["rank"], e)
            # a stamp can be at most one tick ahead of the tick that waits for it
            assert e["act"] <= e["t"] + 1 and e["grad"] <= e["t"] + 1
    assert outs[1]["status"] == "left after tick 7" and len(outs[1]["log"]) == 8
    # rank 1's last stamp (8) still arrives, so rank 0 runs tick 8 and learns of the departure before tick 9
    assert outs[0]["status"] == "neighbour 1 left before tick 9" and len(outs[0]["log"]) == 9
