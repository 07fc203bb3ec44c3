"""fp64 CPU oracle (test infrastructure only).

Only tests, the smoke check and the bench's CPU-baseline leg may import this
package.  It shares no code with the CUDA library and never imports it.
"""
from .oracle import (build, bucket, forward, forward_one, lib_path, max_threads)  # noqa: F401
