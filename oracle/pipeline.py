"""Pipelined Backpropagation, one tick at a time, on the CPU (test
infrastructure; float64 unless another dtype is asked for).

Follows Appendix "Pipelined Backpropagation": S stages, batch size one, each
stage does one forward and one backward transformation per time step; a sample
entering at tick i is forwarded by stage s at tick i+s, reaches the loss at
tick i+S-1 and is back-propagated by stage s at tick i+2(S-1)-s, so it takes
2S-1 steps and stage s sees D_s = 2(S-1-s) updates between its forward and
its backward on the same sample (Eq. F_i: forward weights w^s_{i-2(S-1-s)}).
The gradient is G(x_i; F_i, W_i): forward with the (predicted) weights of the
forward tick, backward with the weights current at the backward tick.  Every
stage is updated separately with its own delay (Section "Methods").

The program is written per sample: everything a stage produces is stored
under the key (stage, sample id), so a stage can only ever read what an
earlier tick wrote for that sample.

Fill-and-drain mode (`update_size` = N > 0; Section 1 and Appendix
"Pipelined Backpropagation": mini-batch SGD on a pipeline).  N samples enter on
N consecutive ticks, the pipeline then drains for 2(S-1) ticks in which nothing
enters, and only when it is empty are all stages updated, with the mean of the
N gradients and plain SGD with momentum; one update takes N + 2S - 2 ticks.
Every sample then sees the same weights forward and backward, so the result
is ordinary mini-batch SGD with momentum.

Weight stashing (`weight_stash`; Appendix "Pipelined Backpropagation", Eq.
"W_{i+1} = W_i - eta grad L(x_i; F_i)", the PipeDream rule the paper compares
with): every stage keeps the weights it used for a sample's forward pass and
uses those same weights for that sample's backward pass, so the gradient is
the true gradient at F_i; the update still lands on the current weights.
"""
import numpy as np

from . import layers as L
from .optimizer import StageOptimizer

# Operation codes of the layer list (the library's public enumeration).
OP_FC, OP_CONV2D, OP_GROUPNORM, OP_RELU, OP_MAXPOOL, OP_AVGPOOL_GLOBAL, \
    OP_ADD_SKIP, OP_SOFTMAX_CE = range(8)

FLAG_SC, FLAG_LWP, FLAG_LWP_WFORM = 1, 2, 4


class _Stage:
    """One pipeline stage: FC or CONV2D head plus what rides with it."""

    def __init__(self, index):
        self.index = index
        self.head = None          # the FC / CONV2D layer record
        self.gn_groups = 0
        self.skip = None          # (source stage, mode, joins before the normalisation)
        self.relu = False
        self.maxpool = None       # (k, stride, pad)
        self.avgpool = False
        self.loss = False
        self.src = -1             # stage whose output is the input (-1: network input)
        self.in_shape = None
        self.z_shape = None       # shape after head (+GN, skip, ReLU)
        self.out_shape = None
        self.n_params = 0

    # parameter views into one flat vector, in layer order
    def split(self, theta):
        h = self.head
        if h.op == OP_FC:
            nw = h.c_in * h.c_out
            return theta[:nw].reshape(h.c_out, h.c_in), theta[nw:nw + h.c_out], None, None
        nw = h.c_out * h.c_in * h.k * h.k
        W = theta[:nw].reshape(h.c_out, h.c_in, h.k, h.k)
        if self.gn_groups:
            return W, None, theta[nw:nw + h.c_out], theta[nw + h.c_out:nw + 2 * h.c_out]
        return W, None, None, None

    rnd = None                # operand rounding of the convolutions (None or a function)
    margins = False           # record how close the ReLU / max-pool decisions were

    def forward(self, theta_hat, x, skip_in):
        """Returns (stage output, what the backward needs, convolution output after a
        pre-normalisation skip addition: the residual sum later stages may add to theirs)."""
        h = self.head
        W, b, gamma, beta = self.split(theta_hat)
        st = {"x": x}
        res = None
        if h.op == OP_FC:
            n = L.fc_forward(W, b, x.ravel()).reshape(-1, 1, 1)
        else:
            n = L.conv2d_forward(W, x, h.stride, h.pad, self.rnd)
            if self.skip is not None and self.skip[2]:
                # pre-activation residual network: the running sum joins here, before the normalisation
                n = n + L.skip_forward(skip_in, self.skip[1], n.shape)
            res = n
            if self.gn_groups:
                n, st["zhat"], st["rstd"] = L.groupnorm_forward(gamma, beta, n, self.gn_groups)
        if self.skip is not None and not self.skip[2]:
            n = n + L.skip_forward(skip_in, self.skip[1], n.shape)
        st["pre"] = n
        a = L.relu_forward(n) if self.relu else n
        if self.margins:
            # smallest distance of any decision from flipping, relative to the tensor's rms
            rms = float(np.sqrt(np.mean(n * n))) or 1.0
            nz = np.abs(n[n != 0])
            st["margin"] = float(nz.min()) / rms if (self.relu and nz.size) else float("inf")
        if self.maxpool is not None:
            if self.margins:
                a, st["arg"], gap = L.maxpool_forward(a, *self.maxpool, want_gap=True)
                st["margin"] = min(st["margin"], gap / rms)
            else:
                a, st["arg"] = L.maxpool_forward(a, *self.maxpool)
        if self.avgpool:
            a = L.avgpool_forward(a)
        return a, st, res

    def backward(self, theta, st, dy, need_dx, skip_shape, dres=None):
        """Returns (g flat like theta, dx or None, dskip or None).  dres: gradient that later
        stages sent straight to this stage's convolution output (they added it to theirs
        before their normalisation), or None."""
        h = self.head
        W, b, gamma, beta = self.split(theta)
        pre = st["pre"]
        d = dy.reshape(self.out_shape)
        if self.avgpool:
            d = L.avgpool_backward(d, pre.shape[1:])
        if self.maxpool is not None:
            d = L.maxpool_backward(st["arg"], d, pre.shape[1:])
        if self.relu:
            d = L.relu_backward(pre, d)
        dskip = None
        if self.skip is not None and not self.skip[2]:
            dskip = L.skip_backward(d, self.skip[1], skip_shape)
        g = np.zeros_like(theta)
        if h.op == OP_FC:
            dx, gW, gb = L.fc_backward(W, st["x"].ravel(), d.ravel())
            nw = gW.size
            g[:nw] = gW.ravel()
            g[nw:] = gb
            dx = dx.reshape(st["x"].shape) if need_dx else None
        else:
            nw = W.size
            if self.gn_groups:
                d, gg, gbeta = L.groupnorm_backward(gamma, st["zhat"], st["rstd"], d, self.gn_groups)
                g[nw:nw + h.c_out] = gg
                g[nw + h.c_out:] = gbeta
            if dres is not None:
                d = d + dres
            if self.skip is not None and self.skip[2]:
                dskip = L.skip_backward(d, self.skip[1], skip_shape)
            dx, gW = L.conv2d_backward(W, st["x"], d, h.stride, h.pad, self.rnd)
            g[:nw] = gW.ravel()
            if not need_dx:
                dx = None
        return g, dx, dskip


def build_stages(layer_list, stage_of_layer, in_shape):
    """Group the layer list into stages and infer every shape."""
    stages = []
    for lay, s in zip(layer_list, stage_of_layer):
        op = int(lay.op)
        if op in (OP_FC, OP_CONV2D):
            if s != len(stages):
                raise ValueError("a stage must start with its FC/CONV2D layer")
            st = _Stage(s)
            st.head = lay
            st.src = lay.src if lay.src >= 0 else s - 1
            src_shape = tuple(in_shape) if st.src < 0 else stages[st.src].out_shape
            st.in_shape = src_shape
            if op == OP_FC:
                if int(np.prod(src_shape)) != lay.c_in:
                    raise ValueError("FC input size mismatch at stage %d" % s)
                st.z_shape = (lay.c_out, 1, 1)
                st.n_params = lay.c_in * lay.c_out + lay.c_out
            else:
                if src_shape[0] != lay.c_in:
                    raise ValueError("conv channel mismatch at stage %d" % s)
                oh = L.conv_out_size(src_shape[1], lay.k, lay.stride, lay.pad)
                ow = L.conv_out_size(src_shape[2], lay.k, lay.stride, lay.pad)
                st.z_shape = (lay.c_out, oh, ow)
                st.n_params = lay.c_out * lay.c_in * lay.k * lay.k
            st.out_shape = st.z_shape
            stages.append(st)
            continue
        st = stages[s]
        if op == OP_GROUPNORM:
            st.gn_groups = lay.groups
            st.n_params += 2 * st.head.c_out
        elif op == OP_ADD_SKIP:
            st.skip = (lay.src, lay.skip_mode & 1, bool(lay.skip_mode & 2))
            if st.skip[2] and (st.head.op != OP_CONV2D or stages[lay.src].head.op != OP_CONV2D):
                raise ValueError("a pre-normalisation skip joins two convolution stages")
        elif op == OP_RELU:
            st.relu = True
        elif op == OP_MAXPOOL:
            st.maxpool = (lay.k, lay.stride, lay.pad)
            c, h, w = st.z_shape
            st.out_shape = (c, L.conv_out_size(h, lay.k, lay.stride, lay.pad),
                            L.conv_out_size(w, lay.k, lay.stride, lay.pad))
        elif op == OP_AVGPOOL_GLOBAL:
            st.avgpool = True
            st.out_shape = (st.z_shape[0], 1, 1)
        elif op == OP_SOFTMAX_CE:
            st.loss = True
        else:
            raise ValueError("unknown op %d" % op)
    return stages


class PBOracle:
    """PB + SC + LWP on a layer list; `tick` advances the pipeline one step."""

    def __init__(self, layer_list, stage_of_layer, in_shape, n_classes, lr,
                 momentum, flags=FLAG_SC | FLAG_LWP, dtype=np.float64,
                 sc_delay_scale=1, horizon_scale=1, record=False, conv_operands=None,
                 margins=False, update_size=0, weight_stash=False):
        """conv_operands: None, or "bf16" to round both operands of every
        convolution product (forward, data gradient, weight gradient) to
        bfloat16 while accumulating in `dtype`.  margins: log in
        `self.min_margin[(stage, sample)]` how close that forward's ReLU /
        max-pool decisions came to flipping (relative to the tensor's rms)."""
        self.dtype = dtype
        self.stages = build_stages(layer_list, stage_of_layer, in_shape)
        for st in self.stages:
            st.rnd = L.round_bf16 if conv_operands == "bf16" else None
            st.margins = margins
        self.min_margin = {}
        self.S = len(self.stages)
        if not self.stages[-1].loss:
            raise ValueError("the last stage must end in SOFTMAX_CE")
        self.in_shape = tuple(in_shape)
        self.update_size = int(update_size)
        if self.update_size > 0:
            flags = 0           # no delay between a sample's forward and backward weights: nothing to compensate
        self.cycle = self.update_size + 2 * (self.S - 1)     # ticks per update when filling and draining
        self.gsum = None
        self.lr, self.m, self.flags = lr, momentum, flags
        self.sc_delay_scale, self.horizon_scale = sc_delay_scale, horizon_scale
        self.n_params = sum(st.n_params for st in self.stages)
        self.opt = None
        self.t = 0
        self.out, self.stash, self.dsum, self.labels = {}, {}, {}, {}
        self.res, self.dres = {}, {}      # residual sums (forward) and the gradients sent straight to them (backward)
        self.res_sources = {st.skip[0] for st in self.stages if st.skip is not None and st.skip[2]}
        self.weight_stash = bool(weight_stash)
        self.wstash = {}          # (stage, sample) -> weights of that sample's forward pass
        self.record = record
        self.fwd_version, self.bwd_version, self.grads = {}, {}, {}
        self.history = [[] for _ in self.stages]   # (w, v) after each version
        self.last_logits = None   # logits behind the most recent loss (for error scaling in tests)

    def delay(self, s):
        """D_s = 2 (S - 1 - s): updates between stage s's forward and backward."""
        return 2 * (self.S - 1 - s)

    def set_weights(self, flat):
        flat = np.asarray(flat)
        assert flat.size == self.n_params
        self.opt, off = [], 0
        for st in self.stages:
            D = self.delay(st.index)
            self.opt.append(StageOptimizer(
                flat[off:off + st.n_params], self.lr, self.m, D,
                use_sc=bool(self.flags & FLAG_SC), use_lwp=bool(self.flags & FLAG_LWP),
                w_form=bool(self.flags & FLAG_LWP_WFORM),
                sc_delay=self.sc_delay_scale * D, horizon=self.horizon_scale * D,
                dtype=self.dtype))
            off += st.n_params
            if self.record:
                self.history[st.index].append((self.opt[-1].w.copy(), self.opt[-1].v.copy()))

    def set_mitigation(self, sc_delay_scale, horizon_scale):
        """Stage s uses the SC coefficients of delay sc_delay_scale * D_s and the
        horizon T = horizon_scale * D_s from the next tick on."""
        self.sc_delay_scale, self.horizon_scale = sc_delay_scale, horizon_scale
        for st, op in zip(self.stages, self.opt):
            D = self.delay(st.index)
            op.set_mitigation(sc_delay_scale * D, horizon_scale * D)

    def load_state(self, flat_w, flat_v):
        """Overwrites every stage's weights and velocities (flat vectors in
        layer order) without touching the pipeline: samples in flight keep what
        they stored.  Bookkeeping only; used to start a tick from a given state."""
        off = 0
        for st, op in zip(self.stages, self.opt):
            op.w = np.array(flat_w[off:off + st.n_params], dtype=self.dtype)
            op.v = np.array(flat_v[off:off + st.n_params], dtype=self.dtype)
            off += st.n_params

    def get_weights(self):
        return np.concatenate([o.w for o in self.opt])

    def get_velocity(self):
        return np.concatenate([o.v for o in self.opt])

    def live(self, i):
        """Did a sample enter at tick i?  Always (i >= 0) in PB; when filling
        and draining only during the first N ticks of a cycle."""
        if i < 0:
            return False
        return self.update_size == 0 or i % self.cycle < self.update_size

    def tick(self, x, label):
        """One time step with new sample (x, label).  Returns the loss the
        last stage computed this tick (sample t-(S-1)), NaN while filling.
        Samples are named by the tick at which they entered; in fill-and-drain
        mode the (x, label) of a draining tick is ignored."""
        S, t = self.S, self.t
        if self.live(t):
            self.out[(-1, t)] = np.asarray(x, dtype=self.dtype).reshape(self.in_shape)
            self.labels[t] = int(label)

        # 1. predicted weights from the state left by the previous tick
        theta_hat = [o.predicted() for o in self.opt]

        # 2. forward of sample t-s at stage s
        for st in self.stages:
            s, i = st.index, t - st.index
            if not self.live(i):
                continue
            skip_in = None
            if st.skip is not None:
                skip_in = (self.res if st.skip[2] else self.out)[(st.skip[0], i)]
            y, stash, res = st.forward(theta_hat[s], self.out[(st.src, i)], skip_in)
            self.out[(s, i)], self.stash[(s, i)] = y, stash
            if s in self.res_sources:
                self.res[(s, i)] = res
            if self.weight_stash:
                self.wstash[(s, i)] = theta_hat[s]
            if st.margins:
                self.min_margin[(s, i)] = stash["margin"]
            if self.record:
                self.fwd_version[(s, i)] = self.opt[s].version

        # 3. loss and its gradient at the last stage (same tick: delay 0)
        loss = float("nan")
        i = t - (S - 1)
        if self.live(i):
            self.last_logits = self.out[(S - 1, i)].ravel().copy()
            loss, delta = L.softmax_ce(self.out[(S - 1, i)].ravel(), self.labels.pop(i))
            self.dsum[(S - 1, i)] = delta.reshape(-1, 1, 1)

        # 4. backward of sample t-2(S-1)+s at stage s, with the current weights
        grads = {}
        for st in self.stages:
            s, j = st.index, t - 2 * (S - 1) + st.index
            if not self.live(j):
                continue
            dy = self.dsum.pop((s, j))
            skip_shape = None
            if st.skip is not None:
                src_stage = self.stages[st.skip[0]]
                skip_shape = src_stage.z_shape if st.skip[2] else src_stage.out_shape
            theta_b = self.wstash.pop((s, j)) if self.weight_stash else self.opt[s].w
            g, dx, dskip = st.backward(theta_b, self.stash.pop((s, j)), dy,
                                       st.src >= 0, skip_shape, self.dres.pop((s, j), None))
            if dx is not None:
                self._accumulate((st.src, j), dx)
            if dskip is not None:
                if st.skip[2]:
                    key = (st.skip[0], j)
                    self.dres[key] = self.dres[key] + dskip if key in self.dres else dskip
                else:
                    self._accumulate((st.skip[0], j), dskip)
            self.res.pop((s, j), None)
            grads[s] = g
            del self.out[(s, j)]
            if s == 0:
                del self.out[(-1, j)]
            if self.record:
                self.bwd_version[(s, j)] = self.opt[s].version
                self.grads[(s, j)] = g.copy()

        # 5. update every stage that received a gradient
        if self.update_size > 0:
            # fill and drain: gradients wait until the pipeline is empty, then every
            # stage takes one SGDM step with their mean
            if self.gsum is None:
                self.gsum = [np.zeros_like(o.w) for o in self.opt]
            for s, g in grads.items():
                self.gsum[s] = self.gsum[s] + g
            if t % self.cycle == self.cycle - 1:
                for s in range(S):
                    self.opt[s].update(self.gsum[s] / self.dtype(self.update_size))
                self.gsum = None
            self.t += 1
            return loss
        for s, g in grads.items():
            self.opt[s].update(g)
            if self.record:
                self.history[s].append((self.opt[s].w.copy(), self.opt[s].v.copy()))
        self.t += 1
        return loss

    def _accumulate(self, key, d):
        if key in self.dsum:
            self.dsum[key] = self.dsum[key] + d
        else:
            self.dsum[key] = d
