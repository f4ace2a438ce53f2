"""Stored oracle outputs (tests/golden/oracle_cases.txt, written by tests/golden/make_golden.py from the
oracle alone): the oracle must still return them, and so must the CUDA path."""
import os
import sys

import numpy as np
import pytest

import oracle

sys.path.insert(0, os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden"))
import make_golden  # noqa: E402

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "oracle_cases.txt")


def stored():
    out = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        label, n, rest = (x.strip() for x in line.split("|"))
        bits, t, prof = rest.split()
        out[(label, int(n[2:]))] = (int(bits, 16), int(t), bytes.fromhex(prof))
    return out


def compare(label, wl, p, c, t, want):
    for n in range(wl.N):
        bits, tt, prof = want[(label, n)]
        assert int(np.asarray(c)[n:n + 1].view(np.uint32)[0]) == bits, (label, n)
        assert int(t[n]) == tt and np.asarray(p)[n].tobytes() == prof, (label, n)


def test_oracle_still_returns_the_stored_values():
    want = stored()
    count = 0
    for label, wl in make_golden.cases():
        p, c, t = oracle.solve_batch(wl.errors, wl.times, wl.B)
        compare(label, wl, p, c, t, want)
        count += wl.N
    assert count == len(want)


@pytest.mark.gpu
@pytest.mark.parametrize("fmt", [1, 2])
def test_cuda_path_returns_the_stored_values(fmt):
    import torch

    from paper_2201_13096_b200 import binding

    want = stored()
    for label, wl in make_golden.cases():
        plan = binding.Plan(wl.times, wl.B, device=0, table_format=fmt)
        p, c, t = binding.solve_batch(plan, torch.from_numpy(wl.errors).cuda())
        torch.cuda.synchronize()
        plan.check_status()
        compare(label, wl, p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy(), want)
        plan.close()
