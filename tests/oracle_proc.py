"""The CPU checker in a process of its own.

The full-size ResNet-50 comparisons run two or three instances of the checker
(float64, float32, without operand rounding) next to the engine; each takes
about a second per tick, so they run side by side in spawned processes (spawn,
not fork: the parent holds a CUDA context).  `RemoteOracle` has the few calls
the comparison loop needs; all arithmetic stays in `oracle/`."""
import multiprocessing as mp

import numpy as np


def _serve(conn, wl, dtype_name, kw):
    import os
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    if root not in sys.path:
        sys.path.insert(0, root)
    from tests.parity import make_oracle
    o = make_oracle(wl, dtype=np.dtype(dtype_name).type, **kw)
    while True:
        msg = conn.recv()
        op = msg[0]
        if op == "tick":
            with np.errstate(all="ignore"):
                loss = o.tick(msg[1], msg[2])
            mxl = float(np.abs(o.last_logits).max()) if o.last_logits is not None else 0.0
            conn.send((loss, mxl))
        elif op == "state":
            conn.send((o.get_weights(), o.get_velocity(), [p.version for p in o.opt]))
        elif op == "mitigation":
            o.set_mitigation(*msg[1])
            conn.send(None)
        elif op == "close":
            conn.close()
            return


# Several instances run side by side, each with its own BLAS thread pool: unbounded pools
# oversubscribe the cores (busy-waiting threads) and make every instance many times slower.
MAX_SIDE_BY_SIDE = 3
_THREAD_VARS = ("OMP_NUM_THREADS", "OPENBLAS_NUM_THREADS", "MKL_NUM_THREADS")


class RemoteOracle:
    def __init__(self, wl, dtype=np.float64, **kw):
        import os
        ctx = mp.get_context("spawn")
        self.conn, child = ctx.Pipe()
        self.proc = ctx.Process(target=_serve, args=(child, wl, np.dtype(dtype).name, kw), daemon=True)
        threads = str(max(1, ((os.cpu_count() or 4) - 1) // MAX_SIDE_BY_SIDE))
        saved = {v: os.environ.get(v) for v in _THREAD_VARS}
        os.environ.update({v: threads for v in _THREAD_VARS})      # inherited by the spawned interpreter
        try:
            self.proc.start()
        finally:
            for v, old in saved.items():
                if old is None:
                    os.environ.pop(v, None)
                else:
                    os.environ[v] = old
        child.close()
        self.last_max_logit = 0.0

    def tick_begin(self, x, y):
        self.conn.send(("tick", np.asarray(x), int(y)))

    def tick_end(self):
        loss, self.last_max_logit = self.conn.recv()
        return loss

    def state(self):
        self.conn.send(("state",))
        return self.conn.recv()

    def set_mitigation(self, *scales):
        self.conn.send(("mitigation", scales))
        self.conn.recv()

    def close(self):
        try:
            self.conn.send(("close",))
        except (OSError, BrokenPipeError):
            pass
        self.proc.join(timeout=10)
        if self.proc.is_alive():
            self.proc.kill()
