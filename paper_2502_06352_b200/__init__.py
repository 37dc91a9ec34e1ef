"""Relaxed (LANTERN++) tree verification on B200: CUDA kernels behind a C ABI.

p is the DRAFTER distribution and q the TARGET distribution, as in the paper.
Every function here only marshals arguments for liblantern.so; all arithmetic
runs in the CUDA kernels.  Importing fails loudly if the library is missing.
"""
from .binding import (  # noqa: F401
    LIB_PATH,
    LanternError,
    Params,
    Tree,
    Forest,
    build_neighbors,
    save_neighbors,
    load_neighbors,
    sample_draft_tree,
    verify_tree,
    verify_tree_static,
    philox_raw,
    set_cluster_size,
    verify_tree_path,
    sample_draft_tree_path,
    DraftPool,
    expand_frontier,
    trim_tree,
    lib,
)
