"""CPU oracle (test infrastructure only).

Only tests, the smoke check and the benchmark's cpu_baseline / reference legs may
import this package.  The CUDA library never does.
"""
from .ps_oracle import (  # noqa: F401
    Oracle,
    OracleConfig,
    build_oracle,
    build_tree,
    gumbel_sample,
    num_threads,
    philox4x32,
    row_stats,
    set_threads,
    uniforms,
    verify,
    verify_tree,
)
