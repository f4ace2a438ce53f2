"""CPU oracle of the SPDY dynamic program.  Test infrastructure: only tests, the smoke check and
the benchmark's CPU-baseline leg may import this package; the CUDA product path never does."""
from .spdy_ref import build, solve_batch, last_row, lib_path  # noqa: F401
