"""The allocation-free entry point against the ordinary engine and the CPU checker.

Some users of this library run where device memory may not be allocated (a
fixed memory budget, or inside another framework's allocator); for them
pb_mlp_run_static keeps all of its scratch in a static array inside the
library.  It must give the numbers pb_create + pb_run give, also when the
array still holds an earlier call's contents; it must match the CPU checker
like every other path; and the amount of free device memory must be the same
after a call as before it."""
import numpy as np
import pytest

from pb_workloads import he_normal_weights, make_inputs, mlp

pytestmark = pytest.mark.gpu

TOL = 1e-4


def _engine_reference(wl, x, y, n):
    import torch
    from tests.parity import make_engine
    eng = make_engine(wl)
    xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    losses = torch.zeros(n, device="cuda")
    eng.run(xd, yd, n, losses)
    eng.sync()
    out = losses.cpu().numpy(), eng.get_weights(), eng.get_velocity()
    eng.destroy()
    return out


def _static_run(wl, sizes, x, y, n):
    import torch
    import paper_2003_11666_b200 as p
    w = torch.from_numpy(he_normal_weights(wl.seed, wl)).cuda()
    v = torch.zeros_like(w)
    xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    losses = torch.full((n,), 7.0, device="cuda")
    p.mlp_run_static(sizes, wl.lr, wl.momentum, wl.flags, w, v, xd, yd, n, losses,
                     stream=torch.cuda.current_stream().cuda_stream)
    return losses.cpu().numpy(), w.cpu().numpy(), v.cpu().numpy()


def _close(a, b):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    return np.linalg.norm(a - b) <= TOL * max(np.linalg.norm(b), 1e-12)


def test_static_entry_point_matches_engine_on_two_calls_in_a_row():
    sizes_a, sizes_b = [64, 48, 32, 6], [50, 33, 20, 17, 5]
    for sizes, n in ((sizes_a, 40), (sizes_b, 31)):     # second call: other shapes over the dirty array
        wl = mlp(sizes, lr=0.003, seed=5)
        x, y = make_inputs(wl.seed, n, wl.sample_elems, wl.n_classes)
        ref_l, ref_w, ref_v = _engine_reference(wl, x, y, n)
        got_l, got_w, got_v = _static_run(wl, sizes, x, y, n)
        S = wl.n_stages
        assert np.isnan(got_l[:S - 1]).all()
        assert _close(got_l[S - 1:], ref_l[S - 1:])
        assert _close(got_w, ref_w) and _close(got_v, ref_v)
    # and the very same problem again gives the very same answer
    wl = mlp(sizes_a, lr=0.003, seed=5)
    x, y = make_inputs(wl.seed, 40, wl.sample_elems, wl.n_classes)
    a = _static_run(wl, sizes_a, x, y, 40)
    b = _static_run(wl, sizes_a, x, y, 40)
    for u, v in zip(a, b):
        np.testing.assert_array_equal(u, v)


def test_static_entry_point_matches_the_cpu_checker_and_allocates_nothing():
    import torch
    from tests.parity import compare_state, make_oracle, tensor_slices
    sizes, n = [72, 40, 24, 7], 36
    wl = mlp(sizes, lr=0.003, seed=7)
    x, y = make_inputs(wl.seed, n, wl.sample_elems, wl.n_classes)
    o = make_oracle(wl)
    ref_l = np.array([o.tick(x[t], y[t]) for t in range(n)])
    # the first call on a device looks up the array's address (and loads the kernels);
    # free memory is compared across the calls after it
    _static_run(wl, sizes, x, y, 4)
    import paper_2003_11666_b200 as p
    w0 = he_normal_weights(wl.seed, wl)
    w = torch.from_numpy(w0).cuda()
    v = torch.zeros_like(w)
    xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    losses = torch.full((n,), 7.0, device="cuda")
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    p.mlp_run_static(sizes, wl.lr, wl.momentum, wl.flags, w, v, xd, yd, n, losses,
                     stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "the call changed the free device memory by %d bytes" % (free_before - free_after)
    got_l = losses.cpu().numpy().astype(np.float64)
    S = wl.n_stages
    assert np.isnan(got_l[:S - 1]).all()
    assert np.abs(got_l[S - 1:] - ref_l[S - 1:]).max() <= TOL * np.abs(ref_l[S - 1:]).max()
    _, _, fails = compare_state(tensor_slices(o), w0, w.cpu().numpy(), v.cpu().numpy(), o.get_weights(), o.get_velocity(),
                                [op.version for op in o.opt], TOL, TOL)
    assert not fails, fails


def test_static_entry_point_rejects_what_does_not_fit():
    import torch
    import paper_2003_11666_b200 as p
    sizes = [2048] * 13 + [10]      # rings and gradient hand-off rows of this net need well over 4 MiB
    n_par = sum(a * b + b for a, b in zip(sizes[:-1], sizes[1:]))
    w = torch.zeros(n_par, device="cuda")
    v = torch.zeros_like(w)
    xd = torch.zeros(2, 2048, device="cuda")
    yd = torch.zeros(2, dtype=torch.int32, device="cuda")
    with pytest.raises(p.PBError) as e:
        p.mlp_run_static(sizes, 0.01, 0.9, 3, w, v, xd, yd, 2)
    assert e.value.code == -1 and "scratch" in str(e.value)
    with pytest.raises(p.PBError):
        p.mlp_run_static([8], 0.01, 0.9, 3, w, v, xd, yd, 2)            # no layer
    with pytest.raises(p.PBError):
        p.mlp_run_static([8, 4], 0.01, 0.9, 8, w, v, xd, yd, 2)         # flag outside SC|LWP
