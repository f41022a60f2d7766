"""Layer mathematics for the CPU checker (test infrastructure; float64).

The paper trains standard networks (Section 2.1 groups "convolution,
normalization, and ReLU into one stage"; Experiment Details: Group
Normalization replaces Batch Normalization) and does not restate their layer
equations, so each function below is the textbook definition written out
directly: no im2col, no blocking, loops where the definition has sums over
small index sets and one matrix product per kernel offset for the channel sum.

All tensors of one sample are [C, H, W]; conv weights are [C_out, C_in, k, k];
FC weights are [out, in].
"""
import numpy as np

GN_EPS = 1e-5


# ---------------------------------------------------------------- fully connected
def fc_forward(W, b, x):
    return W @ x + b


def fc_backward(W, x, dy):
    """Returns (dx, gW, gb) for y = W x + b."""
    return W.T @ dy, np.outer(dy, x), dy.copy()


# ---------------------------------------------------------------- convolution
def _pad(x, pad):
    if pad == 0:
        return x
    return np.pad(x, ((0, 0), (pad, pad), (pad, pad)))


def conv_out_size(n, k, stride, pad):
    return (n + 2 * pad - k) // stride + 1


def round_bf16(x):
    """Round to the nearest bfloat16 (ties to even) and return in x's dtype:
    the value is first taken to float32, whose upper 16 bits are a bfloat16."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((b >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    b = (b + r) & np.uint32(0xFFFF0000)
    return b.view(np.float32).astype(x.dtype)


def conv2d_forward(W, x, stride, pad, rnd=None):
    """z[o, p, q] = sum_{c, r, s} W[o, c, r, s] * xpad[c, p*stride + r, q*stride + s].
    `rnd`, if given, is applied to both operands first (reduced-precision
    multiplicands with exact products and wide accumulation)."""
    if rnd is not None:
        W, x = rnd(W), rnd(x)
    co, ci, k, _ = W.shape
    oh = conv_out_size(x.shape[1], k, stride, pad)
    ow = conv_out_size(x.shape[2], k, stride, pad)
    xp = _pad(x, pad)
    z = np.zeros((co, oh, ow), dtype=x.dtype)
    for r in range(k):
        for s in range(k):
            win = xp[:, r:r + stride * oh:stride, s:s + stride * ow:stride]
            z += np.tensordot(W[:, :, r, s], win, axes=([1], [0]))
    return z


def conv2d_backward(W, x, dz, stride, pad, rnd=None):
    """Returns (dx, gW) of conv2d_forward; `rnd` as there, on W, x and dz."""
    if rnd is not None:
        W, x, dz = rnd(W), rnd(x), rnd(dz)
    co, ci, k, _ = W.shape
    oh, ow = dz.shape[1], dz.shape[2]
    xp = _pad(x, pad)
    dxp = np.zeros_like(xp)
    gW = np.zeros_like(W)
    for r in range(k):
        for s in range(k):
            sl = (slice(None), slice(r, r + stride * oh, stride),
                  slice(s, s + stride * ow, stride))
            gW[:, :, r, s] = np.tensordot(dz, xp[sl], axes=([1, 2], [1, 2]))
            dxp[sl] += np.tensordot(W[:, :, r, s], dz, axes=([0], [0]))
    if pad:
        dxp = dxp[:, pad:-pad, pad:-pad]
    return dxp, gW


# ---------------------------------------------------------------- group normalisation
def groupnorm_forward(gamma, beta, z, groups):
    """Per group of C/groups channels: zhat = (z - mean) / sqrt(var + eps) with
    the biased variance over the group's channels and pixels; n = gamma*zhat + beta.
    Returns (n, zhat, rstd[groups])."""
    c, h, w = z.shape
    zg = z.reshape(groups, -1)
    mean = zg.mean(axis=1, keepdims=True)
    var = ((zg - mean) ** 2).mean(axis=1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + z.dtype.type(GN_EPS))
    zhat = ((zg - mean) * rstd).reshape(c, h, w)
    n = gamma[:, None, None] * zhat + beta[:, None, None]
    return n, zhat, rstd[:, 0]


def groupnorm_backward(gamma, zhat, rstd, dn, groups):
    """Returns (dz, g_gamma, g_beta)."""
    c, h, w = zhat.shape
    g_gamma = (dn * zhat).sum(axis=(1, 2))
    g_beta = dn.sum(axis=(1, 2))
    dzhat = (dn * gamma[:, None, None]).reshape(groups, -1)
    zh = zhat.reshape(groups, -1)
    m1 = dzhat.mean(axis=1, keepdims=True)
    m2 = (dzhat * zh).mean(axis=1, keepdims=True)
    dz = rstd[:, None] * (dzhat - m1 - zh * m2)
    return dz.reshape(c, h, w), g_gamma, g_beta


# ---------------------------------------------------------------- pointwise / pooling
def relu_forward(x):
    return np.where(x > 0, x, x.dtype.type(0))


def relu_backward(x_pre, dy):
    """Derivative taken as 0 at x = 0."""
    return np.where(x_pre > 0, dy, dy.dtype.type(0))


def maxpool_forward(x, k, stride, pad, want_gap=False):
    """Returns (y, arg) where arg[c, p, q] is the flat index (row*W + col in
    the unpadded input) of the first maximum in row-major window order;
    padding never wins.  With want_gap also returns the smallest distance
    between the largest and second largest entry over windows whose maximum
    is positive (how close any window came to choosing differently)."""
    c, h, w = x.shape
    oh = conv_out_size(h, k, stride, pad)
    ow = conv_out_size(w, k, stride, pad)
    y = np.full((c, oh, ow), -np.inf, dtype=x.dtype)
    second = np.full((c, oh, ow), -np.inf, dtype=x.dtype)
    arg = np.full((c, oh, ow), -1, dtype=np.int64)
    for p in range(oh):
        for q in range(ow):
            for r in range(k):
                for s in range(k):
                    ih, iw = p * stride + r - pad, q * stride + s - pad
                    if 0 <= ih < h and 0 <= iw < w:
                        v = x[:, ih, iw]
                        better = v > y[:, p, q]
                        second[:, p, q] = np.where(better, y[:, p, q], np.maximum(second[:, p, q], v))
                        y[better, p, q] = v[better]
                        arg[better, p, q] = ih * w + iw
    if want_gap:
        pos = y > 0
        gap = float((y - second)[pos].min()) if pos.any() else float("inf")
        return y, arg, gap
    return y, arg


def maxpool_backward(arg, dy, in_hw):
    c = dy.shape[0]
    h, w = in_hw
    dx = np.zeros((c, h * w), dtype=dy.dtype)
    for ch in range(c):
        np.add.at(dx[ch], arg[ch].ravel(), dy[ch].ravel())
    return dx.reshape(c, h, w)


def avgpool_forward(x):
    return x.mean(axis=(1, 2)).reshape(-1, 1, 1)


def avgpool_backward(dy, in_hw):
    h, w = in_hw
    return np.broadcast_to(dy.reshape(-1, 1, 1) / (h * w), (dy.shape[0], h, w)).copy()


def skip_forward(x, mode, out_shape):
    """mode 0: identity.  mode 1: keep every second pixel in each direction and
    append zero channels up to out_shape[0] (parameter-free shortcut)."""
    if mode == 0:
        return x
    c = x.shape[0]
    y = np.zeros(out_shape, dtype=x.dtype)
    y[:c] = x[:, ::2, ::2]
    return y


def skip_backward(dy, mode, in_shape):
    if mode == 0:
        return dy.copy()
    dx = np.zeros(in_shape, dtype=dy.dtype)
    dx[:, ::2, ::2] = dy[:in_shape[0]]
    return dx


# ---------------------------------------------------------------- loss
def softmax_ce(o, label):
    """loss = logsumexp(o) - o[label] (natural log, max subtracted);
    delta = softmax(o) - onehot(label)."""
    mx = o.max()
    e = np.exp(o - mx)
    s = e.sum()
    loss = np.log(s) + mx - o[label]
    delta = e / s
    delta[label] -= 1.0
    return loss, delta
