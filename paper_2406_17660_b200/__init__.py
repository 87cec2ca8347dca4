"""GRASS structured-sparse gradient step for B200: Python binding over the C-ABI library.

The CUDA library (libgrass_b200.so, built by `python -m paper_2406_17660_b200.build`)
does all the work; this package only marshals torch tensors into pointers.
Importing the package does not load the library; the first call does, and
raises if it has not been built.
"""
from .binding import (  # noqa: F401
    GrassError, BF16, F32, SEL_TOPR, SEL_MULTINOMIAL_NORM, SEL_MULTINOMIAL_NORM2, SEL_UNIFORM,
    SEL_MULTINOMIAL_NORM_NR, SEL_MULTINOMIAL_NORM2_NR, SEL_UNIFORM_NR,
    grass_row_norms, grass_select, grass_select_static, grass_select_workspace_bytes,
    grass_project_grad, grass_project_workspace_bytes,
    grass_grad_row_norms, grass_grad_row_norms_workspace_bytes,
    grass_subspace_adam, grass_adam_scatter, grass_adam_scatter_batched,
    grass_project_grad_batched, grass_project_batched_workspace_bytes,
    grass_project_grad_ex, grass_project_plan, ProjectOpts, GATHER_AUTO, GATHER_PREPASS, GATHER_IN_CTA,
    GATHER_COOPERATIVE, PAIR_AUTO, PAIR_NEVER, PAIR_ALWAYS, grass_scatter_update, grass_scatter_update_cols, grass_device_status,
    grass_status_string, grass_profile_begin, grass_profile_end, grass_profile_end_timeline, grass_selftest_bounded_wait, library_path, load_library,
)
from .step import GrassLayer  # noqa: F401
