"""Seeded synthetic inputs for the quantized-Adam parameter-server step.

This package only describes parameter-set shapes and draws random tensors from
stated distributions.  It contains none of the optimizer's or the quantizers'
arithmetic, so the CPU oracle and the CUDA path can both consume what it makes.
"""
from .shapes import resnet18_shapes, bert_base_shapes, numel
from .workloads import Workload, get_workload, WORKLOAD_NAMES
from .generate import gradients, initial_weights

__all__ = [
    "resnet18_shapes", "bert_base_shapes", "numel",
    "Workload", "get_workload", "WORKLOAD_NAMES",
    "gradients", "initial_weights",
]
