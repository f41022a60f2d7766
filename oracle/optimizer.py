"""Per-stage optimizer: SGD with momentum, Spike Compensation, Linear Weight
Prediction and their combination.  Test infrastructure; float64.

Notation follows the paper's Methods section: weights w, velocity v, momentum
m, learning rate eta, delay D, spike coefficients a and b, horizon T.
"""
import numpy as np


def sc_coefficients(m, D):
    """Default Spike Compensation coefficients SC_D (Eq. "a = m^D and
    b = (1 - m^D)/(1 - m)"): b is the sum of the D momentum terms the delayed
    gradient missed, a the decay the no-delay impulse response has reached."""
    a = m ** D
    b = float(D) if m == 1.0 else (1.0 - m ** D) / (1.0 - m)
    return a, b


class StageOptimizer:
    """State (w, v) of one stage and the paper's update rules.

    use_sc   -> a, b = SC_D coefficients for delay `sc_delay`; else a=1, b=0,
                which is plain SGDM (Eqs. v_{t+1} = m v_t + g_t,
                w_{t+1} = w_t - eta v_{t+1}).
    use_lwp  -> horizon T = `horizon`; else T = 0.
    w_form   -> predict with the weight-difference form
                w + T (w - w_prev) instead of the velocity form w - eta T v.
    """

    def __init__(self, w, lr, m, delay, use_sc=True, use_lwp=True,
                 w_form=False, sc_delay=None, horizon=None, dtype=np.float64):
        self.dtype = dtype
        self.w = np.array(w, dtype=dtype).copy()
        self.v = np.zeros_like(self.w)
        self.w_prev = self.w.copy()
        self.lr, self.m, self.delay = dtype(lr), dtype(m), int(delay)
        sc_delay = delay if sc_delay is None else sc_delay
        horizon = delay if horizon is None else horizon
        if use_sc:
            a, b = sc_coefficients(float(m), sc_delay)
        else:
            a, b = 1.0, 0.0
        self.a, self.b = dtype(a), dtype(b)
        self.T = dtype(horizon if use_lwp else 0)
        self.w_form = bool(w_form)
        self.use_sc, self.use_lwp = bool(use_sc), bool(use_lwp)
        self.version = 0        # number of updates applied so far

    def set_mitigation(self, sc_delay, horizon):
        """Other compensation strengths from now on (generalized Spike
        Compensation with the coefficients of another delay, e.g. SC_2D;
        Appendix "Extended Weight Prediction Horizons": T = alpha D).  The
        state (w, v) is untouched: the next prediction uses the new T, the
        next update the new a, b."""
        if self.use_sc:
            a, b = sc_coefficients(float(self.m), sc_delay)
            self.a, self.b = self.dtype(a), self.dtype(b)
        if self.use_lwp:
            self.T = self.dtype(horizon)

    def predicted(self):
        """Weights the forward pass uses (Eq. "LWP velocity form":
        w_hat = w - eta T v; weight-difference form: w + T (w - w_prev)),
        from the state as it stands now."""
        if self.w_form:
            return self.w + self.T * (self.w - self.w_prev)
        return self.w - self.lr * self.T * self.v

    def update(self, g):
        """Combined mitigation step (Section "Combined Mitigation"):
        v <- m v + g ;  w <- w - eta (a v + b g)."""
        g = np.asarray(g, dtype=self.dtype)
        self.w_prev = self.w.copy()
        self.v = self.m * self.v + g
        self.w = self.w - self.lr * (self.a * self.v + self.b * g)
        self.version += 1
