"""CPU oracle for relaxed (LANTERN++) tree verification.  TEST INFRASTRUCTURE.

Plain, slow, double-precision numpy code that follows the paper step by step.
It shares nothing with the CUDA path: no kernels, headers, tables or helpers.
Only the tests, the smoke check and the timed CPU baseline of the benchmark may
import it; the product never does.

Notation (Sec. 2, "Notations"): p is the DRAFTER distribution, q the TARGET
distribution; the acceptance ratio is q / p.

Pinned by tests/test_oracle_*.py against closed forms, brute force and special
cases.  Parity with numbers printed in the paper is unpinned: every number in
its tables needs trained models and captions that are not available.
"""

from .postprocess import fma_f32, combine_f32, postprocess_row  # noqa: F401
from .neighbors import neighbor_table, neighbor_row  # noqa: F401
from .tree import tree_children  # noqa: F401
from .verify import relaxed_mass, moved_mass, sibling_loop, inverse_cdf, verify_node, verify_sequence, walk, verify_batch  # noqa: F401
from .sampler import sample_children, sample_draft_tree  # noqa: F401
from .philox import philox4x32_10, uniform_open, uniform_halfopen, stream_uniforms  # noqa: F401
from .dynamic_tree import top_children, expand_frontier, trim, breadth_first, draft_dynamic_tree  # noqa: F401
