"""B200-native Pipelined Backpropagation engine (CUDA library + thin binding).

`PB` wraps one engine handle; see include/pb.h for the meaning of each call.
The package never computes on the CPU: without the built shared library the
binding raises.
"""
from .binding import PB, PBError, mlp_run_static, split_plan, bench_l2_bandwidth, bench_fp32_fma, PB_SC, PB_LWP, PB_LWP_WFORM, PB_CONV_BF16, PB_WEIGHT_STASH, load_library, LIB_PATH, EXPORTS

__all__ = ["PB", "PBError", "mlp_run_static", "split_plan", "bench_l2_bandwidth", "bench_fp32_fma", "PB_SC", "PB_LWP", "PB_LWP_WFORM", "PB_CONV_BF16", "PB_WEIGHT_STASH", "load_library",
           "LIB_PATH", "EXPORTS"]
