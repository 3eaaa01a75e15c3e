"""B200-native GDN tree verification and commit (Section 3.4 of "Trees from Marginals").

``gdn_tree_verify`` and ``gdn_tree_commit`` are thin bindings over the C-ABI CUDA library built from ``csrc/``;
``synth`` holds the seeded synthetic workload generators.  There is no CPU fallback: every call raises if the CUDA
library has not been built.
"""
from . import synth  # noqa: F401
from .binding import (  # noqa: F401
    GdnShape,
    gdn_status_string,
    gdn_tree_commit,
    gdn_tree_commit_host,
    gdn_tree_commit_padded,
    gdn_tree_commit_verify,
    gdn_tree_commit_verify_padded,
    gdn_tree_commit_verify_host,
    gdn_tree_commit_verify_host_arena_bytes,
    gdn_tree_host_arena_bytes,
    gdn_tree_plan,
    gdn_tree_plan_bytes,
    gdn_tree_validate_host,
    gdn_tree_verify,
    gdn_tree_verify_host,
    gdn_tree_verify_padded,
    gdn_tree_verify_planned,
    gdn_tree_verify_recurrent,
    gdn_tree_verify_static,
    gdn_tree_workspace_bytes,
    library_path,
    load_library,
)
