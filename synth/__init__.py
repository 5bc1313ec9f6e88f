"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests.

This package draws random numbers and lists workload shapes.  It holds none of the
method's arithmetic: no sign unpacking, no scaling, no matrix product, no device layout.
"""
from .workloads import (  # noqa: F401
    LayerInputs,
    LayerShape,
    CONFIG0_SHAPE,
    llama2_7b_layer_shapes,
    llama3_8b_layer_shapes,
    llama_70b_layer_shapes,
    make_layer,
    make_x,
    make_planes_constant,
    fp16_bits,
)
