"""Worker of the two-rank CPU test of the stage split: every rank asks the library for the
plan, then the ranks run the hand-off protocol of include/pb.h on the host - after tick t a
rank stamps t + 1 at its neighbours, before tick t it needs both of its own stamps at t -
with keys of the rendezvous store in place of peer stores.  One rank leaves early (between ticks,
announcing it in the store); the other must notice before its next tick instead of waiting."""
import json
import os
import sys
import time

import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import paper_2003_11666_b200 as pbm  # noqa: E402
from pb_workloads import mlp  # noqa: E402


def main():
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    store = dist.distributed_c10d._get_default_store()
    wl = mlp([2048] * 6 + [10])
    plan = pbm.split_plan(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, world)
    plans = [None] * world
    dist.all_gather_object(plans, plan)
    lo, hi = plan[rank]
    prev_r, next_r = (rank - 1 if rank > 0 else None), (rank + 1 if rank + 1 < world else None)
    stamps = {"act": 0, "grad": 0}            # what the neighbours have delivered so far
    n_ticks, leave_at = 12, 7                 # the last rank leaves after tick `leave_at`
    log, status = [], "ok"
    def wait_stamp(key, src, t):
        """The bounded wait of a tick, on the host: the neighbour's stamp reaches t, or the store
        says that the neighbour has left (then nothing is launched any more), or a second passes."""
        t0 = time.time()
        while time.time() - t0 < 1.0 + 29.0 * (t == 1):      # (the first exchange also covers process start-up)
            if store.check([key]):
                v = int(store.get(key))
                if v >= t:
                    return v
            if store.check(["left%d" % src]):
                return None
            time.sleep(0.002)
        return -1

    for t in range(n_ticks):
        # the wait of tick t: both stamps must have reached t
        gone = None
        if prev_r is not None and t > 0:
            v = wait_stamp("act_stamp_of_%d" % rank, prev_r, t)
            gone = prev_r if v is None else gone
            stamps["act"] = stamps["act"] if v is None else v
        if gone is None and next_r is not None and t > 0:
            v = wait_stamp("grad_stamp_of_%d" % rank, next_r, t)
            gone = next_r if v is None else gone
            stamps["grad"] = stamps["grad"] if v is None else v
        if gone is not None:
            status = "neighbour %d left before tick %d" % (gone, t)
            break
        ok = (prev_r is None or stamps["act"] >= t) and (next_r is None or stamps["grad"] >= t)
        log.append({"t": t, "act": stamps["act"], "grad": stamps["grad"], "ok": ok})
        # ... the tick itself would run here; then the stamps go into the neighbours' memory
        # (here: keys of the store, written like the plain peer stores of the GPU code) ...
        if next_r is not None:
            store.set("act_stamp_of_%d" % next_r, str(t + 1))
        if prev_r is not None:
            store.set("grad_stamp_of_%d" % prev_r, str(t + 1))
        if rank == world - 1 and t == leave_at:
            store.set("left%d" % rank, "1")       # leaves between ticks, after its last stamp
            status = "left after tick %d" % t
            break
    with open(os.path.join(sys.argv[1], "split_rank%d.json" % rank), "w") as f:
        json.dump({"rank": rank, "plan": plan, "plans_equal": all(p == plan for p in plans), "range": [lo, hi],
                   "log": log, "status": status}, f)
    # no barrier: a rank that has left does not come back; leave the group without it
    # (the last stamp of each rank has no reader any more and is not waited for)
    os._exit(0)


if __name__ == "__main__":
    main()
