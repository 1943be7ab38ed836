"""TEST INFRASTRUCTURE: fp64 CPU oracle of Gram-threshold selection.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this
package.  It shares nothing with the CUDA library.
"""
from .ada_oracle import (  # noqa: F401
    build, normalize, select_full, full_rows, cascade_step, op_count,
    jaccard, turnover, tau_update, nearest, attention_reps, num_threads, set_threads, CascadeResult,
)
