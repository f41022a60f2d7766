"""Stage split (several ranks, each running a contiguous range of stages and handing the
boundary activation forward and the boundary gradient backward) against the CPU checker.
Run here on ONE device: the ranks' handles are ticked in turn on one stream, so every
tick stamp is in place before it is looked at and no kernel ever waits for another."""
import numpy as np
import pytest

from pb_workloads import he_normal_weights, make_inputs, mlp
from tests.parity import compare_state, make_oracle, tensor_slices

pytestmark = pytest.mark.gpu

TOL = 1e-4


def _ranks(wl, n_ranks):
    import torch
    from paper_2003_11666_b200 import PB
    st = torch.cuda.current_stream().cuda_stream
    engs = [PB(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, wl.lr, wl.momentum, wl.flags,
               stream=st, rank=r, n_ranks=n_ranks) for r in range(n_ranks)]
    ports = [e.split_ports() for e in engs]
    for r, e in enumerate(engs):
        e.split_connect(ports[r - 1] if r > 0 else None, ports[r + 1] if r + 1 < n_ranks else None)
        e.set_weights(he_normal_weights(wl.seed, wl))
    return engs


@pytest.mark.parametrize("sizes,n_ranks,flags", [([48, 40, 33, 24, 16, 5], 2, 3), ([48, 40, 33, 24, 16, 5], 3, 3),
                                                  ([64, 64, 48, 32, 6], 4, 3), ([40, 33, 24, 5], 2, 0),
                                                  ([130, 260, 131, 70, 3], 2, 7)])
def test_split_pipeline_matches_checker(sizes, n_ranks, flags):
    import torch
    from paper_2003_11666_b200 import split_plan
    wl = mlp(sizes, lr=0.003, seed=41, flags=flags)
    S = wl.n_stages
    plan = split_plan(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, n_ranks)
    assert plan[0][0] == 0 and plan[-1][1] == S and all(a[1] == b[0] for a, b in zip(plan, plan[1:]))
    engs = _ranks(wl, n_ranks)
    assert [e.split_range() for e in engs] == plan
    o = make_oracle(wl)
    slices = tensor_slices(o)
    w_init = he_normal_weights(wl.seed, wl)
    n = 2 * (S - 1) + 20
    x, y = make_inputs(wl.seed, n, wl.sample_elems, wl.n_classes)
    xd = torch.from_numpy(x).cuda()
    for t in range(n):
        lo = o.tick(x[t], y[t])
        lg = None
        for r, e in enumerate(engs):             # rank 0 first: the order in which nothing waits
            last = r == n_ranks - 1
            l = e.tick(xd[t] if r == 0 else None, int(y[t]), want_loss=last)
            lg = l if last else lg
        if np.isnan(lo):
            assert np.isnan(lg)
        else:
            assert abs(lg - lo) <= TOL * max(abs(lo), float(np.abs(o.last_logits).max()))
        if t % 3 == 0 or t == n - 1:
            gw = sum(e.get_weights() for e in engs)          # every rank returns zeros for the others' stages
            gv = sum(e.get_velocity() for e in engs)
            _, _, fails = compare_state(slices, w_init, gw, gv, o.get_weights(), o.get_velocity(),
                                        [p.version for p in o.opt], TOL, TOL)
            assert not fails, "tick %d: %s" % (t, "; ".join(fails[:4]))
    assert min(p.version for p in o.opt) >= 20
    for e in engs:
        e.destroy()


def test_split_agrees_with_the_unsplit_engine_to_rounding():
    # same kernels; only the row bands of the blocks differ (each handle balances its own stages),
    # and with them the grouping of the partial sums of W^T delta: agreement to float32 rounding
    import torch
    from tests.parity import make_engine
    wl = mlp([96, 80, 64, 48, 7], lr=0.002, seed=42)
    n = 40
    x, y = make_inputs(wl.seed, n, wl.sample_elems, wl.n_classes)
    xd = torch.from_numpy(x).cuda()
    whole = make_engine(wl)
    engs = _ranks(wl, 2)
    for t in range(n):
        a = whole.tick(xd[t], int(y[t]))
        engs[0].tick(xd[t], int(y[t]), want_loss=False)
        b = engs[1].tick(None, int(y[t]))
        assert (np.isnan(a) and np.isnan(b)) or abs(a - b) <= 1e-5 * max(1.0, abs(a))
    gw, gv = sum(e.get_weights() for e in engs), sum(e.get_velocity() for e in engs)
    assert np.linalg.norm(whole.get_weights() - gw) <= 1e-5 * np.linalg.norm(gw - he_normal_weights(wl.seed, wl))
    assert np.linalg.norm(whole.get_velocity() - gv) <= 1e-5 * np.linalg.norm(gv)
    whole.destroy()
    for e in engs:
        e.destroy()


def test_split_handles_refuse_what_they_cannot_do():
    import torch
    from paper_2003_11666_b200 import PB, PBError
    from pb_workloads import tiny_cnn
    st = torch.cuda.current_stream().cuda_stream
    wl = tiny_cnn()
    with pytest.raises(PBError) as e:
        PB(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, wl.lr, wl.momentum, wl.flags, stream=st, rank=0, n_ranks=2)
    assert e.value.code == -6                                   # convolutional networks are not split
    wl = mlp([16, 12, 8, 4])
    with pytest.raises(PBError):
        PB(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, wl.lr, wl.momentum, wl.flags, stream=st, rank=2, n_ranks=2)
    with pytest.raises(PBError):
        PB(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, wl.lr, wl.momentum, wl.flags, stream=st, rank=0, n_ranks=9)
    a = PB(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, wl.lr, wl.momentum, wl.flags, stream=st, rank=0, n_ranks=2)
    a.set_weights(he_normal_weights(wl.seed, wl))
    x = torch.zeros(16, device="cuda")
    with pytest.raises(PBError) as e:
        a.tick(x, 0)                                            # not connected to its neighbour yet: nothing is launched
    assert e.value.code == -1 and a.tick_count == 0
    with pytest.raises(PBError):
        a.split_connect(None, None)                             # rank 0 of 2 has a next rank
    a.destroy()
