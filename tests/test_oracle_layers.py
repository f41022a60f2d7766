"""Pins for the checker's layer mathematics: brute-force loops, central finite
differences in float64 and torch CPU autograd.  CPU only."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import layers as L


def _fd(f, x, eps=1e-6):
    """Central finite-difference gradient of scalar f at x."""
    g = np.zeros_like(x)
    it = np.nditer(x, flags=["multi_index"])
    for _ in it:
        i = it.multi_index
        old = x[i]
        x[i] = old + eps
        fp = f()
        x[i] = old - eps
        fm = f()
        x[i] = old
        g[i] = (fp - fm) / (2 * eps)
    return g


@pytest.mark.parametrize("k,stride,pad,h", [(3, 1, 1, 6), (3, 2, 1, 7), (1, 2, 0, 6), (7, 2, 3, 12), (1, 1, 0, 5)])
def test_conv_forward_bruteforce_and_torch(k, stride, pad, h):
    rng = np.random.default_rng(k * 10 + stride)
    ci, co, w = 3, 4, h + 1
    x = rng.standard_normal((ci, h, w))
    W = rng.standard_normal((co, ci, k, k))
    z = L.conv2d_forward(W, x, stride, pad)
    oh, ow = z.shape[1:]
    ref = np.zeros_like(z)
    for o in range(co):
        for p in range(oh):
            for q in range(ow):
                acc = 0.0
                for c in range(ci):
                    for r in range(k):
                        for s in range(k):
                            ih, iw = p * stride + r - pad, q * stride + s - pad
                            if 0 <= ih < h and 0 <= iw < w:
                                acc += W[o, c, r, s] * x[c, ih, iw]
                ref[o, p, q] = acc
    np.testing.assert_allclose(z, ref, rtol=1e-12, atol=1e-12)
    zt = F.conv2d(torch.tensor(x)[None], torch.tensor(W), stride=stride, padding=pad)[0].numpy()
    np.testing.assert_allclose(z, zt, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("k,stride,pad", [(3, 1, 1), (3, 2, 1), (1, 2, 0)])
def test_conv_backward_finite_differences(k, stride, pad):
    rng = np.random.default_rng(3)
    x = rng.standard_normal((2, 5, 6))
    W = rng.standard_normal((3, 2, k, k))
    z = L.conv2d_forward(W, x, stride, pad)
    c = rng.standard_normal(z.shape)       # loss = sum(c * z)
    dx, gW = L.conv2d_backward(W, x, c, stride, pad)
    f = lambda: float((c * L.conv2d_forward(W, x, stride, pad)).sum())
    np.testing.assert_allclose(dx, _fd(f, x), rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(gW, _fd(f, W), rtol=1e-6, atol=1e-7)


def test_groupnorm_against_torch_and_fd():
    rng = np.random.default_rng(4)
    c, groups = 6, 3
    z = rng.standard_normal((c, 4, 5)) * 2 + 0.7
    gamma, beta = rng.standard_normal(c), rng.standard_normal(c)
    n, zhat, rstd = L.groupnorm_forward(gamma, beta, z, groups)
    zt = torch.tensor(z, requires_grad=True)
    gt, bt = torch.tensor(gamma, requires_grad=True), torch.tensor(beta, requires_grad=True)
    nt = F.group_norm(zt[None], groups, gt, bt, eps=1e-5)[0]
    np.testing.assert_allclose(n, nt.detach().numpy(), rtol=1e-12, atol=1e-12)
    cot = rng.standard_normal(n.shape)
    (nt * torch.tensor(cot)).sum().backward()
    dz, gg, gb = L.groupnorm_backward(gamma, zhat, rstd, cot, groups)
    np.testing.assert_allclose(dz, zt.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(gg, gt.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(gb, bt.grad.numpy(), rtol=1e-10, atol=1e-12)
    f = lambda: float((cot * L.groupnorm_forward(gamma, beta, z, groups)[0]).sum())
    np.testing.assert_allclose(dz, _fd(f, z), rtol=1e-5, atol=1e-7)
    # unit statistics per group: mean 0, biased variance 1 - eps*rstd^2
    zg = zhat.reshape(groups, -1)
    np.testing.assert_allclose(zg.mean(1), 0, atol=1e-12)
    np.testing.assert_allclose((zg ** 2).mean(1), 1 - 1e-5 * rstd ** 2, rtol=1e-10)


@pytest.mark.parametrize("k,stride,pad,h", [(2, 2, 0, 6), (3, 2, 1, 7), (3, 2, 1, 8)])
def test_maxpool_against_torch(k, stride, pad, h):
    rng = np.random.default_rng(5)
    x = rng.standard_normal((3, h, h + 1))
    y, arg = L.maxpool_forward(x, k, stride, pad)
    xt = torch.tensor(x, requires_grad=True)
    yt = F.max_pool2d(xt[None], k, stride, pad)[0]
    np.testing.assert_array_equal(y, yt.detach().numpy())
    cot = rng.standard_normal(y.shape)
    (yt * torch.tensor(cot)).sum().backward()
    np.testing.assert_allclose(L.maxpool_backward(arg, cot, x.shape[1:]), xt.grad.numpy(),
                               rtol=0, atol=1e-15)


def test_maxpool_tie_goes_to_first_in_window_order():
    x = np.zeros((1, 2, 2))
    y, arg = L.maxpool_forward(x, 2, 2, 0)
    assert y[0, 0, 0] == 0 and arg[0, 0, 0] == 0
    x[0, 1, 0] = x[0, 0, 1] = 3.0
    _, arg = L.maxpool_forward(x, 2, 2, 0)
    assert arg[0, 0, 0] == 1          # (row 0, col 1) comes before (row 1, col 0)


def test_relu_derivative_zero_at_zero():
    x = np.array([-1.0, 0.0, 2.0])
    np.testing.assert_array_equal(L.relu_forward(x), [0, 0, 2])
    np.testing.assert_array_equal(L.relu_backward(x, np.ones(3)), [0, 0, 1])


def test_avgpool_and_skip():
    rng = np.random.default_rng(6)
    x = rng.standard_normal((4, 6, 6))
    y = L.avgpool_forward(x)
    np.testing.assert_allclose(y.ravel(), x.reshape(4, -1).mean(1))
    d = rng.standard_normal((4, 1, 1))
    np.testing.assert_allclose(L.avgpool_backward(d, (6, 6)).sum(axis=(1, 2)), d.ravel())
    s = L.skip_forward(x, 1, (8, 3, 3))
    np.testing.assert_array_equal(s[:4], x[:, ::2, ::2])
    assert not s[4:].any()
    dy = rng.standard_normal((8, 3, 3))
    dx = L.skip_backward(dy, 1, (4, 6, 6))
    # adjoint identity <skip(x), dy> == <x, skip^T(dy)>
    assert float((s * dy).sum()) == pytest.approx(float((x * dx).sum()), rel=1e-12)
    assert L.skip_forward(x, 0, x.shape) is x


def test_softmax_ce_against_torch_and_extremes():
    rng = np.random.default_rng(7)
    o = rng.standard_normal(10) * 3
    loss, delta = L.softmax_ce(o.copy(), 4)
    ot = torch.tensor(o, requires_grad=True)
    lt = F.cross_entropy(ot[None], torch.tensor([4]))
    lt.backward()
    assert loss == pytest.approx(lt.item(), rel=1e-12)
    np.testing.assert_allclose(delta, ot.grad.numpy(), rtol=1e-12, atol=1e-15)
    assert delta.sum() == pytest.approx(0, abs=1e-14)
    # uniform logits: loss = ln(n); huge logits stay finite
    assert L.softmax_ce(np.zeros(1000), 7)[0] == pytest.approx(np.log(1000), rel=1e-13)
    big, _ = L.softmax_ce(np.array([1e4, 0.0, -1e4]), 1)
    assert big == pytest.approx(1e4, rel=1e-12)


def test_fc_backward_fd():
    rng = np.random.default_rng(8)
    W, b, x = rng.standard_normal((4, 5)), rng.standard_normal(4), rng.standard_normal(5)
    c = rng.standard_normal(4)
    dx, gW, gb = L.fc_backward(W, x, c)
    f = lambda: float(c @ L.fc_forward(W, b, x))
    np.testing.assert_allclose(dx, _fd(f, x), rtol=1e-7, atol=1e-9)
    np.testing.assert_allclose(gW, _fd(f, W), rtol=1e-7, atol=1e-9)
    np.testing.assert_allclose(gb, _fd(f, b), rtol=1e-7, atol=1e-9)


def test_round_bf16_matches_torch_and_ties_to_even():
    rng = np.random.default_rng(9)
    x = np.concatenate([rng.standard_normal(5000) * 10.0 ** rng.integers(-6, 6, 5000),
                        [0.0, -0.0, 1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -7, -1.0 - 2 ** -8]])
    got = L.round_bf16(x)
    ref = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(got, ref)
    # 1 + 2^-8 lies half-way between 1 and 1 + 2^-7: the even mantissa (1.0) wins;
    # 1 + 3*2^-8 lies half-way between 1 + 2^-7 and 1 + 2^-6: the even one is 1 + 2^-6
    assert L.round_bf16(np.array([1.0 + 2 ** -8]))[0] == 1.0
    assert L.round_bf16(np.array([1.0 + 3 * 2 ** -8]))[0] == 1.0 + 2 ** -6
    assert got.dtype == x.dtype


def test_conv_with_rounded_operands_is_conv_of_rounded_operands():
    rng = np.random.default_rng(10)
    x, W = rng.standard_normal((3, 6, 6)), rng.standard_normal((4, 3, 3, 3))
    dz = rng.standard_normal((4, 3, 3))
    z = L.conv2d_forward(W, x, 2, 1, L.round_bf16)
    zt = F.conv2d(torch.tensor(L.round_bf16(x))[None], torch.tensor(L.round_bf16(W)), stride=2, padding=1)[0]
    np.testing.assert_allclose(z, zt.numpy(), rtol=1e-12, atol=1e-12)
    dx, gW = L.conv2d_backward(W, x, dz, 2, 1, L.round_bf16)
    dx0, gW0 = L.conv2d_backward(L.round_bf16(W), L.round_bf16(x), L.round_bf16(dz), 2, 1)
    np.testing.assert_array_equal(dx, dx0)
    np.testing.assert_array_equal(gW, gW0)
    assert np.abs(z - L.conv2d_forward(W, x, 2, 1)).max() > 1e-4


def test_maxpool_gap_reports_the_closest_call():
    x = np.array([[[1.0, 0.5, 3.0, 2.75], [0.25, 0.0, 1.0, 0.0]]])
    y, arg, gap = L.maxpool_forward(x, 2, 2, 0, want_gap=True)
    np.testing.assert_array_equal(y[0, 0], [1.0, 3.0])
    assert gap == 0.25
    _, _, gap0 = L.maxpool_forward(np.zeros((1, 2, 2)), 2, 2, 0, want_gap=True)
    assert gap0 == float("inf")          # no positive maximum: nothing can flip a gradient
