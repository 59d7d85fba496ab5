"""CPU oracle for the PaFu-KV hot path.  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It shares no code with the CUDA library and neither imports the other.
"""
from .pafu_oracle import (  # noqa: F401
    build, score, select, compact, cache_update, attention, sse, sse_mean_first, sse_cols, sse_global_max, sse_global_avg, n_threads,
)
