"""Seeded synthetic workloads shared by the tests, the benchmark and both implementations.

This package holds network tables (lists of layer descriptors), the counter-based
random streams and the input / initial-weight generators.  It contains none of the
method's arithmetic: no forward, backward, optimiser, partition or snapshot code.
"""
from .nets import (Layer, KIND, ACT, har_cnn, mobilenetv2, vgg16, tiny_mbv2, tiny_vgg, continual_mbv2,
                   param_shapes, state_shapes, num_units, config)
from .inputs import rng_stream, make_batch, init_params, init_state, flat_unit_params

__all__ = ["Layer", "KIND", "ACT", "har_cnn", "mobilenetv2", "vgg16", "tiny_mbv2", "tiny_vgg", "continual_mbv2",
           "param_shapes", "state_shapes", "num_units", "config", "rng_stream", "make_batch",
           "init_params", "init_state", "flat_unit_params"]
