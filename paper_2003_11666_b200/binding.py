"""ctypes binding of libpb_b200.so: argument marshalling only.

Every function here has the name and meaning of the C entry point it calls
(include/pb.h).  Nothing is computed on the Python side and there is no
fallback: if the shared library is missing or fails to load, importing the
handle class raises.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpb_b200.so")

PB_SC, PB_LWP, PB_LWP_WFORM, PB_CONV_BF16, PB_WEIGHT_STASH = 1, 2, 4, 8, 16

EXPORTS = [
    "pb_create", "pb_set_weights", "pb_tick", "pb_run", "pb_run_host", "pb_get_weights",
    "pb_get_velocity", "pb_sync", "pb_num_params", "pb_num_stages", "pb_stage_delay",
    "pb_tick_count", "pb_last_launch_count", "pb_device_bytes", "pb_profile_enable",
    "pb_profile_ms", "pb_last_error", "pb_destroy", "pb_mlp_run_static", "pb_set_mitigation",
    "pb_set_update_size", "pb_kernel_min_bytes", "pb_bench_l2_bandwidth", "pb_bench_fp32_fma",
    "pb_split_plan", "pb_create_split", "pb_split_range", "pb_split_ports", "pb_split_connect",
]


class pb_layer(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("op", "c_in", "c_out", "k", "stride", "pad", "groups", "src", "skip_mode")]


class pb_split_port(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("act", "act_stamp", "grad", "grad_stamp")]


class PBError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("pb error %d: %s" % (code, msg))
        self.code = code


_lib = None


def load_library():
    """Loads the shared library (building is a separate, explicit step)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError("%s is missing: run `python -m paper_2003_11666_b200.build` "
                          "(the engine has no CPU fallback)" % LIB_PATH)
    lib = C.CDLL(LIB_PATH)
    vp, i32, f32 = C.c_void_p, C.c_int, C.c_float
    lib.pb_create.argtypes = [C.POINTER(pb_layer), i32, C.POINTER(C.c_int32), i32, i32, i32, i32,
                              f32, f32, C.c_uint, vp, C.POINTER(vp)]
    lib.pb_set_weights.argtypes = [vp, vp, C.c_size_t]
    lib.pb_set_mitigation.argtypes = [vp, f32, f32]
    lib.pb_set_update_size.argtypes = [vp, i32]
    lib.pb_tick.argtypes = [vp, vp, i32, C.POINTER(f32)]
    lib.pb_run.argtypes = [vp, vp, vp, i32, vp]
    lib.pb_run_host.argtypes = [vp, vp, vp, i32, vp]
    lib.pb_get_weights.argtypes = [vp, vp, C.c_size_t]
    lib.pb_get_velocity.argtypes = [vp, vp, C.c_size_t]
    lib.pb_sync.argtypes = [vp]
    lib.pb_num_params.argtypes = [vp]
    lib.pb_num_params.restype = C.c_size_t
    lib.pb_num_stages.argtypes = [vp]
    lib.pb_stage_delay.argtypes = [vp, i32]
    lib.pb_tick_count.argtypes = [vp]
    lib.pb_tick_count.restype = C.c_longlong
    lib.pb_last_launch_count.argtypes = [vp]
    lib.pb_last_launch_count.restype = C.c_longlong
    lib.pb_device_bytes.argtypes = [vp]
    lib.pb_device_bytes.restype = C.c_size_t
    lib.pb_profile_enable.argtypes = [vp, i32]
    lib.pb_profile_ms.argtypes = [vp, i32, C.POINTER(C.c_longlong)]
    lib.pb_profile_ms.restype = C.c_double
    lib.pb_last_error.argtypes = [vp]
    lib.pb_last_error.restype = C.c_char_p
    lib.pb_destroy.argtypes = [vp]
    lib.pb_destroy.restype = None
    lib.pb_kernel_min_bytes.argtypes = [vp, i32]
    lib.pb_kernel_min_bytes.restype = C.c_double
    lib.pb_bench_l2_bandwidth.argtypes = [C.c_size_t, i32, vp, C.POINTER(C.c_double)]
    lib.pb_bench_fp32_fma.argtypes = [i32, vp, C.POINTER(C.c_double)]
    lib.pb_split_plan.argtypes = [C.POINTER(pb_layer), i32, C.POINTER(C.c_int32), i32, i32, i32, i32, i32,
                                  C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.pb_create_split.argtypes = [C.POINTER(pb_layer), i32, C.POINTER(C.c_int32), i32, i32, i32, i32,
                                    f32, f32, C.c_uint, vp, i32, i32, C.POINTER(vp)]
    lib.pb_split_range.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.pb_split_ports.argtypes = [vp, C.POINTER(pb_split_port)]
    lib.pb_split_connect.argtypes = [vp, C.POINTER(pb_split_port), C.POINTER(pb_split_port)]
    lib.pb_mlp_run_static.argtypes = [C.POINTER(C.c_int32), i32, f32, f32, C.c_uint, vp, vp, vp, vp, i32, vp, vp]
    _lib = lib
    return lib


def _ptr(a):
    """Address of a numpy array, a torch tensor or a raw integer address."""
    if a is None:
        return None
    if isinstance(a, int):
        return a
    if isinstance(a, np.ndarray):
        return a.ctypes.data
    return a.data_ptr()     # torch.Tensor


def mlp_run_static(sizes, lr, momentum, flags, dev_w, dev_v, dev_xs, dev_labels, n_ticks,
                   dev_losses=None, stream=0):
    """pb_mlp_run_static: PB ticks of a small MLP without any device allocation
    (for callers that may not allocate: the scratch is a static array in the
    library).  All tensors are device memory owned by the caller."""
    lib = load_library()
    arr = (C.c_int32 * len(sizes))(*[int(s) for s in sizes])
    rc = lib.pb_mlp_run_static(arr, len(sizes), float(lr), float(momentum), int(flags), _ptr(dev_w),
                               _ptr(dev_v), _ptr(dev_xs), _ptr(dev_labels), int(n_ticks),
                               _ptr(dev_losses), C.c_void_p(stream))
    if rc != 0:
        raise PBError(rc, lib.pb_last_error(None).decode())


def _layer_arrays(layers, stage_of_layer):
    arr = (pb_layer * len(layers))()
    for q, L in enumerate(layers):
        arr[q] = pb_layer(*L.astuple()) if hasattr(L, "astuple") else pb_layer(*L)
    st = (C.c_int32 * len(layers))(*[int(s) for s in stage_of_layer])
    return arr, st


def split_plan(layers, stage_of_layer, in_shape, n_classes, n_ranks):
    """pb_split_plan: [(lo, hi)] stage ranges of the ranks (host arithmetic only)."""
    lib = load_library()
    arr, st = _layer_arrays(layers, stage_of_layer)
    lo, hi = (C.c_int32 * n_ranks)(), (C.c_int32 * n_ranks)()
    rc = lib.pb_split_plan(arr, len(layers), st, int(in_shape[0]), int(in_shape[1]), int(in_shape[2]),
                           int(n_classes), int(n_ranks), lo, hi)
    if rc != 0:
        raise PBError(rc, lib.pb_last_error(None).decode())
    return [(int(a), int(b)) for a, b in zip(lo, hi)]


def bench_l2_bandwidth(nbytes, iters=200, stream=0):
    """pb_bench_l2_bandwidth: GB/s (read + write) of an in-place sweep over `nbytes`."""
    lib = load_library()
    out = C.c_double(0.0)
    rc = lib.pb_bench_l2_bandwidth(int(nbytes), int(iters), C.c_void_p(stream), C.byref(out))
    if rc != 0:
        raise PBError(rc, lib.pb_last_error(None).decode())
    return out.value


def bench_fp32_fma(iters=4096, stream=0):
    """pb_bench_fp32_fma: float32 FMA rate of the CUDA cores in TFLOP/s."""
    lib = load_library()
    out = C.c_double(0.0)
    rc = lib.pb_bench_fp32_fma(int(iters), C.c_void_p(stream), C.byref(out))
    if rc != 0:
        raise PBError(rc, lib.pb_last_error(None).decode())
    return out.value


class PB:
    """Owner of one pb_handle.  Methods mirror the C calls one to one."""

    def __init__(self, layers, stage_of_layer, in_shape, n_classes, lr, momentum,
                 flags=PB_SC | PB_LWP, stream=0, rank=None, n_ranks=None):
        """rank / n_ranks given: pb_create_split (this handle runs one rank's stages)."""
        self._lib = load_library()
        self._h = C.c_void_p()
        arr, st = _layer_arrays(layers, stage_of_layer)
        if n_ranks is None:
            rc = self._lib.pb_create(arr, len(layers), st, int(in_shape[0]), int(in_shape[1]),
                                     int(in_shape[2]), int(n_classes), float(lr), float(momentum),
                                     int(flags), C.c_void_p(stream), C.byref(self._h))
        else:
            rc = self._lib.pb_create_split(arr, len(layers), st, int(in_shape[0]), int(in_shape[1]),
                                           int(in_shape[2]), int(n_classes), float(lr), float(momentum),
                                           int(flags), C.c_void_p(stream), int(rank), int(n_ranks), C.byref(self._h))
        if rc != 0:
            raise PBError(rc, self._lib.pb_last_error(None).decode())
        self.sample_elems = int(in_shape[0]) * int(in_shape[1]) * int(in_shape[2])

    def _check(self, rc):
        if rc != 0:
            raise PBError(rc, self._lib.pb_last_error(self._h).decode())

    def set_weights(self, host_w):
        w = np.ascontiguousarray(host_w, dtype=np.float32)
        self._check(self._lib.pb_set_weights(self._h, w.ctypes.data, w.size))

    def set_mitigation(self, sc_delay_scale, horizon_scale):
        self._check(self._lib.pb_set_mitigation(self._h, float(sc_delay_scale), float(horizon_scale)))

    def set_update_size(self, n_samples):
        self._check(self._lib.pb_set_update_size(self._h, int(n_samples)))

    def tick(self, dev_x, label, want_loss=True):
        loss = C.c_float(float("nan"))
        self._check(self._lib.pb_tick(self._h, _ptr(dev_x), int(label),
                                      C.byref(loss) if want_loss else None))
        return loss.value

    def run(self, dev_xs, dev_labels, n_ticks, dev_losses=None):
        self._check(self._lib.pb_run(self._h, _ptr(dev_xs), _ptr(dev_labels), int(n_ticks),
                                     _ptr(dev_losses)))

    def run_host(self, host_xs, host_labels, n_ticks, host_losses=None):
        self._check(self._lib.pb_run_host(self._h, _ptr(host_xs), _ptr(host_labels), int(n_ticks),
                                          _ptr(host_losses)))

    def get_weights(self):
        out = np.empty(self.num_params, dtype=np.float32)
        self._check(self._lib.pb_get_weights(self._h, out.ctypes.data, out.size))
        return out

    def get_velocity(self):
        out = np.empty(self.num_params, dtype=np.float32)
        self._check(self._lib.pb_get_velocity(self._h, out.ctypes.data, out.size))
        return out

    def sync(self):
        self._check(self._lib.pb_sync(self._h))

    @property
    def num_params(self):
        return int(self._lib.pb_num_params(self._h))

    @property
    def num_stages(self):
        return int(self._lib.pb_num_stages(self._h))

    def stage_delay(self, s):
        return int(self._lib.pb_stage_delay(self._h, int(s)))

    @property
    def tick_count(self):
        return int(self._lib.pb_tick_count(self._h))

    @property
    def last_launch_count(self):
        return int(self._lib.pb_last_launch_count(self._h))

    @property
    def device_bytes(self):
        return int(self._lib.pb_device_bytes(self._h))

    def split_range(self):
        lo, hi = C.c_int32(0), C.c_int32(0)
        self._check(self._lib.pb_split_range(self._h, C.byref(lo), C.byref(hi)))
        return int(lo.value), int(hi.value)

    def split_ports(self):
        port = pb_split_port()
        self._check(self._lib.pb_split_ports(self._h, C.byref(port)))
        return port

    def split_connect(self, prev_rank_port, next_rank_port):
        self._check(self._lib.pb_split_connect(
            self._h, C.byref(prev_rank_port) if prev_rank_port is not None else None,
            C.byref(next_rank_port) if next_rank_port is not None else None))

    def kernel_min_bytes(self, which):
        return float(self._lib.pb_kernel_min_bytes(self._h, int(which)))

    def profile_enable(self, on=True):
        self._check(self._lib.pb_profile_enable(self._h, 1 if on else 0))

    def profile_ms(self, which):
        n = C.c_longlong(0)
        ms = self._lib.pb_profile_ms(self._h, int(which), C.byref(n))
        return float(ms), int(n.value)

    def destroy(self):
        if self._h:
            self._lib.pb_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
