"""Writes tests/golden/oracle_cases.txt: outputs of the CPU oracle on fixed seeded inputs.

The paper prints no worked example of the dynamic program, so these stored values are not the
paper's: they freeze what the pinned oracle returns (a later change to its arithmetic must show up
here and be justified), and give the GPU tests fixed expectations that were never produced by the
CUDA path.  This script calls only `oracle/` and the seeded input generators.

    python tests/golden/make_golden.py
"""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import oracle  # noqa: E402
from paper_2201_13096_b200 import workloads as W  # noqa: E402


def cases():
    for seed in range(8):
        yield f"config0 seed_shift={seed}", W.make_workload(0, seed_shift=seed)
    for seed in (3, 10_003, 17, 10_017):
        yield f"tiny seed={seed} exact={int(seed >= 10_000)} N=3", W.tiny_random_instance(seed, exact=seed >= 10_000, N=3)
    for cfg in (1, 2):
        yield f"config{cfg} N=3", W.make_workload(cfg, N=3)


def main():
    lines = ["# label | per candidate: cost bits (hex) time_used profile (hex bytes)"]
    for label, wl in cases():
        p, c, t = oracle.solve_batch(wl.errors, wl.times, wl.B)
        for n in range(wl.N):
            lines.append(f"{label} | n={n} | {c[n:n + 1].view(np.uint32)[0]:08x} {int(t[n])} {p[n].tobytes().hex()}")
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_cases.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()
