"""Seeded synthetic inputs (model shapes, weights, prompts, tree topologies).

This package holds input generators only: it contains none of the method's
arithmetic and imports neither the CPU oracle nor the CUDA library.  Tests and
the benchmark build inputs here and hand the same tensors to both sides.
"""
from .configs import ModelShape, SHAPES, get_shape  # noqa: F401
from .gen import (  # noqa: F401
    normal_tensor,
    tensor_std,
    uniform_ids,
    weight_specs,
    make_weights,
    make_prompt,
)
from .tree import make_tree, full_tree, chain_tree, TreeTopology  # noqa: F401
