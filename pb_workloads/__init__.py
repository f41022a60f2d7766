"""Seeded synthetic workloads for Pipelined Backpropagation runs.

This package only *describes* problems: it draws inputs, labels and initial
weights from a counter-based generator and lists the layers of the five
benchmark networks.  It holds none of the training arithmetic (no forward,
backward or optimizer math), so both the CPU checker and the CUDA library can
be fed from it without sharing any of the method's code.
"""
from .gen import (splitmix64, uniform01, normal, labels, he_normal_weights,
                  make_inputs)
from .configs import (OP, Layer, Workload, workload, WORKLOAD_NAMES,
                      param_sizes, infer_shapes, work_per_tick, mlp, tiny_cnn, tiny_resnet,
                      tall_bottleneck, tail_cnn, preact_resnet, SKIP_PRENORM)

__all__ = ["splitmix64", "uniform01", "normal", "labels", "he_normal_weights",
           "make_inputs", "OP", "Layer", "Workload", "workload",
           "WORKLOAD_NAMES", "param_sizes", "infer_shapes", "work_per_tick", "mlp", "tiny_cnn",
           "tiny_resnet", "tall_bottleneck", "tail_cnn", "preact_resnet", "SKIP_PRENORM"]
