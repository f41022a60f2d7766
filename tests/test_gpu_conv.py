"""CUDA engine vs CPU checker on convolutional pipelines (through the C ABI)."""
import numpy as np
import pytest

from pb_workloads import tall_bottleneck, tiny_cnn, tiny_resnet, workload
from tests.parity import compare_ticks

pytestmark = pytest.mark.gpu

TOL = 1e-4        # float32 path
TOL_BF16 = 2e-2   # bfloat16 convolution operands, float32 accumulation
# A ReLU / max-pool decision closer to flipping than 2e-6 of the tensor's rms (about
# 30 float32 ulps) can legitimately come out either way in float32; after the first
# one reaches its backward pass the two trajectories may differ by a finite step.
FRAGILE = dict(fragile_margin=2e-6, fragile_tol=5e-3)


@pytest.mark.parametrize("flags", [3, 0, 1, 2])
def test_tiny_cnn(flags):
    wl = tiny_cnn(flags=flags)
    w = compare_ticks(wl, 2 * (wl.n_stages - 1) + 24, TOL)
    assert w["ticks"] == 2 * (wl.n_stages - 1) + 24


def test_tiny_resnet_skips_and_subsampled_shortcut():
    wl = tiny_resnet()
    w = compare_ticks(wl, 2 * (wl.n_stages - 1) + 24, TOL)
    assert w["ticks"] == 2 * (wl.n_stages - 1) + 24


def test_tiny_bottleneck_projection_shortcuts_float32():
    wl = tiny_resnet(bottleneck=True, flags=3)
    w = compare_ticks(wl, 2 * (wl.n_stages - 1) + 24, TOL)
    assert w["ticks"] == 2 * (wl.n_stages - 1) + 24


def test_tiny_bottleneck_bf16_operands():
    wl = tiny_resnet(bottleneck=True, flags=3 | 8)   # bf16 convolution operands
    assert wl.flags & 8
    # The checker rounds the same operands to bfloat16, so the ReLU decisions are taken from
    # equally rounded numbers on both sides.  A float32-level difference in an accumulation
    # can still flip a bfloat16 rounding or a ReLU decision; how far two correct evaluations
    # part is measured by running the checker itself in float32 and float64, and every
    # tensor must stay within max(2e-2, 3 x that distance over its stage and the stages
    # downstream of it).  No fixed looser bound is used.
    w = compare_ticks(wl, 2 * (wl.n_stages - 1) + 24, TOL_BF16, spread_factor=3.0)
    assert w["ticks"] == 2 * (wl.n_stages - 1) + 24
    assert w["min_updates"] >= 24


def test_tall_bf16_net_reaches_the_large_image_paths():
    # 3x256x256 inputs, 8..64 channels: the stem's output has 16384 pixels per channel and the
    # first block's 4096, so this net runs what only large images reach: tensor-core weight
    # gradients that contract over more than 3072 pixels (K sliced, more than three K chunks
    # per slice, so the stage barriers wrap their phase), data gradients with thousands of
    # columns, normalisation groups cut into several pieces per channel, the stem's 3x3/2
    # max-pool backward and its CUDA-core weight gradient over 16384 pixels with bfloat16 operands.
    # Every stage updates from tick 2(S-1)-s on; the window ends 14 ticks after the first one has.
    wl = tall_bottleneck()
    S = wl.n_stages
    n = 2 * (S - 1) + 14
    w = compare_ticks(wl, n, TOL_BF16, spread_factor=3.0, unrounded_loss_tol=TOL_BF16)
    assert w["ticks"] == n and w["min_updates"] >= 14


def test_vgg11_first_64_ticks():
    wl = workload("vgg11")
    w = compare_ticks(wl, 64, TOL, check_every=2, **FRAGILE)
    assert w["ticks"] == 64
    assert w["fragile_tick"] is None or w["fragile_tick"] >= 16   # strict part covers the first updates


def test_resnet20_first_64_ticks_and_first_update_of_every_stage():
    wl = workload("resnet20")
    n = 2 * (wl.n_stages - 1) + 16        # 54: stage 0 first updates at tick 38
    w = compare_ticks(wl, max(n, 64), TOL, check_every=2, **FRAGILE)
    assert w["ticks"] == 64
    assert w["fragile_tick"] is None or w["fragile_tick"] >= 30


def test_resnet50_bf16_first_72_ticks():
    # Full size: 54 stages, 25.6 M parameters, 3x224x224 inputs, bfloat16 convolution
    # operands, literal hyper-parameters.  Losses stay within 2e-2 of the checker (which rounds
    # the same operands to bfloat16); every tensor's displacement and velocity are bounded by
    # 2e-2 or three times the distance between the checker's own float32 and float64 runs
    # (over its stage and the stages downstream), whichever is larger.  The window stops at
    # tick 72: with the literal learning rate the checker's own velocities in stages 36-40
    # pass 1e3 near tick 80 and float32 overflows soon after.  Only stages >= 35 update
    # inside this window; the run below covers the others.
    wl = workload("resnet50")
    w = compare_ticks(wl, 72, TOL_BF16, check_every=4, spread_factor=3.0)
    assert w["ticks"] == 72
    assert w["loss"] <= TOL_BF16


def test_resnet50_bf16_stable_step_every_stage_updates():
    # The same 54 stages at full size with a step size at which the run stays bounded
    # (lr 5e-4; the literal 5e-3 diverges near tick 76), for 2(S-1)+16 = 122 ticks: stage s
    # takes its first update at tick 106-s, so by the end every stage, the stem included, has
    # been compared through at least 16 updates - data and weight gradients of the large
    # feature maps, the sliced tensor-core weight gradients of the first block, the stem's
    # max-pool backward.  The loss is also held to 2e-2 of the checker WITHOUT operand
    # rounding (the paper's arithmetic in float64).
    wl = workload("resnet50")
    wl.lr = 5e-4
    S = wl.n_stages
    n = 2 * (S - 1) + 16
    ticks = set(range(52, n, 6)) | {n - 1}
    w = compare_ticks(wl, n, TOL_BF16, check_ticks=ticks, spread_factor=3.0, unrounded_loss_tol=TOL_BF16,
                      plain_loss_tol=TOL_BF16)
    assert w["ticks"] == n
    assert w["min_updates"] >= 16
    assert w["loss"] <= TOL_BF16


@pytest.mark.parametrize("name,ticks", [("resnet20", 96), ("vgg11", 48)])
def test_two_runs_give_identical_bits(name, ticks):
    # Forward chain, backward chain and FC stage of a tick run on three streams and every
    # reduction has a fixed order: two runs of the same samples must agree bit for bit
    # (a race between the chains, or an atomics-ordered sum, would show up here).
    import torch
    from pb_workloads import make_inputs
    from tests.parity import make_engine
    wl = workload(name)
    x, y = make_inputs(wl.seed, ticks, wl.sample_elems, wl.n_classes)
    xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    outs = []
    for _ in range(2):
        e = make_engine(wl)
        losses = torch.zeros(ticks, device="cuda")
        e.run(xd, yd, ticks, losses)
        e.sync()
        outs.append((losses.cpu().numpy(), e.get_weights(), e.get_velocity()))
        e.destroy()
    S = wl.n_stages
    np.testing.assert_array_equal(outs[0][0][S - 1:], outs[1][0][S - 1:])
    np.testing.assert_array_equal(outs[0][1], outs[1][1])
    np.testing.assert_array_equal(outs[0][2], outs[1][2])
