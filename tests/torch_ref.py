"""A float64 torch (CPU autograd) rendering of a layer list, written without
reference to the checker's code so that the two can be compared in tests."""
import torch
import torch.nn.functional as F

from pb_workloads import OP


class TorchStage:
    def __init__(self, index):
        self.index = index
        self.head = None
        self.gn = 0
        self.skip = None
        self.relu = False
        self.pool = None
        self.avg = False
        self.src = -1
        self.n_params = 0


def build(wl):
    stages = []
    for lay, s in zip(wl.layers, wl.stage_of_layer):
        if lay.op in (OP.FC, OP.CONV2D):
            st = TorchStage(s)
            st.head = lay
            st.src = lay.src if lay.src >= 0 else s - 1
            st.n_params = (lay.c_in * lay.c_out + lay.c_out if lay.op == OP.FC
                           else lay.c_out * lay.c_in * lay.k * lay.k)
            stages.append(st)
        elif lay.op == OP.GROUPNORM:
            stages[s].gn = lay.groups
            stages[s].n_params += 2 * lay.c_out
        elif lay.op == OP.ADD_SKIP:
            stages[s].skip = (lay.src, lay.skip_mode)
        elif lay.op == OP.RELU:
            stages[s].relu = True
        elif lay.op == OP.MAXPOOL:
            stages[s].pool = (lay.k, lay.stride, lay.pad)
        elif lay.op == OP.AVGPOOL_GLOBAL:
            stages[s].avg = True
    return stages


def split(st, theta):
    h = st.head
    if h.op == OP.FC:
        nw = h.c_in * h.c_out
        return theta[:nw].view(h.c_out, h.c_in), theta[nw:], None, None
    nw = h.c_out * h.c_in * h.k * h.k
    W = theta[:nw].view(h.c_out, h.c_in, h.k, h.k)
    if st.gn:
        return W, None, theta[nw:nw + h.c_out], theta[nw + h.c_out:]
    return W, None, None, None


def _mix(value_with_fwd, same_with_bwd):
    """Value of the first argument, derivative of the second."""
    return same_with_bwd + (value_with_fwd - same_with_bwd).detach()


def _shortcut(sk, mode, channels):
    if mode & 1:
        sub = sk[:, ::2, ::2]
        sk = torch.cat([sub, torch.zeros(channels - sub.shape[0], *sub.shape[1:], dtype=sk.dtype)], 0)
    return sk


def stage_forward(st, theta_fwd, x, skip_in, theta_bwd=None):
    """(output, convolution output after a pre-normalisation shortcut) of one stage for input
    x [C,H,W].  With theta_bwd given, values come from theta_fwd while every derivative is taken
    as if the linear maps held theta_bwd (the stored activations stay those of the forward)."""
    tb = theta_fwd if theta_bwd is None else theta_bwd
    Wf, bf, gf, betaf = split(st, theta_fwd)
    Wb, bb, gb, betab = split(st, tb)
    h = st.head
    res = None
    if h.op == OP.FC:
        xf = x.reshape(-1)
        n = _mix(Wf @ xf + bf, Wb @ xf + bb).view(-1, 1, 1)
    else:
        conv = lambda W: F.conv2d(x[None], W, stride=h.stride, padding=h.pad)[0]
        n = _mix(conv(Wf), conv(Wb))
        if st.skip is not None and st.skip[1] & 2:
            n = n + _shortcut(skip_in, st.skip[1], n.shape[0])      # pre-activation network: the running sum
        res = n
        if st.gn:
            zhat = F.group_norm(n[None], st.gn, eps=1e-5)[0]
            n = _mix(gf[:, None, None] * zhat + betaf[:, None, None],
                     gb[:, None, None] * zhat + betab[:, None, None])
    if st.skip is not None and not st.skip[1] & 2:
        n = n + _shortcut(skip_in, st.skip[1], n.shape[0])
    a = F.relu(n) if st.relu else n
    if st.pool is not None:
        k, s, p = st.pool
        a = F.max_pool2d(a[None], k, s, p)[0]
    if st.avg:
        a = a.mean(dim=(1, 2), keepdim=True)
    return a, res


def network_loss(stages, thetas_fwd, x, label, thetas_bwd=None):
    outs, sums = {-1: x}, {}
    for st in stages:
        tb = None if thetas_bwd is None else thetas_bwd[st.index]
        skip_in = None
        if st.skip is not None:
            skip_in = (sums if st.skip[1] & 2 else outs)[st.skip[0]]
        outs[st.index], sums[st.index] = stage_forward(st, thetas_fwd[st.index], outs[st.src], skip_in, tb)
    logits = outs[len(stages) - 1].reshape(1, -1)
    return F.cross_entropy(logits, torch.tensor([int(label)]))
