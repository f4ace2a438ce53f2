"""CPU oracle of the SPDY dynamic program.  Test infrastructure: only tests, the smoke check and
the benchmark's CPU-baseline leg may import this package; the CUDA product path never does."""
from .spdy_ref import build, solve_batch, last_row, lib_path  # noqa: F401
from .spdy_search_ref import (quadratic_errors, time_target, bucketize_times, uniform_profile,  # noqa: F401
                              search)
