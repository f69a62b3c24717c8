"""Seeded synthetic inputs (model shapes, weights, prompts) for the DMTD decode path.

This module holds no arithmetic of the method itself: it only draws random
numbers.  Both the CPU oracle's tests and the CUDA path's tests / benchmark get
their inputs from here, so that neither side depends on the other.
"""
from .shapes import ModelShape, SHAPES, WORKLOADS, Workload
from .weights import make_weights, make_prompts, weight_bytes

__all__ = ["ModelShape", "SHAPES", "WORKLOADS", "Workload", "make_weights",
           "make_prompts", "weight_bytes"]
