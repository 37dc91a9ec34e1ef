"""Seeded synthetic inputs shared by the CPU oracle tests and the CUDA path.

This package only *draws inputs*: tree topologies, logit rows, codebooks and
uniform random numbers.  It contains none of the method's arithmetic (no
softmax, no acceptance rule, no nearest-neighbour search), so that the oracle
and the CUDA kernels can be fed the very same bytes without sharing code.
"""

from .trees import static_tree, tree_levels, TREE_CAPS  # noqa: F401
from .configs import CONFIGS, WorkloadConfig  # noqa: F401
from .generators import (  # noqa: F401
    make_logits,
    make_codebook,
    make_uniforms,
    make_gumbel_uniforms,
    random_sibling_tokens,
    random_neighbor_table,
)
