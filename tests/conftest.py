import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: test needs a CUDA device (sm_100a)")


def load_hand_example():
    """Parse tests/golden/hand_example.txt -> (A, [(alpha, beta, f, S), ...])."""
    import numpy as np
    rows, cases = [], []
    with open(os.path.join(ROOT, "tests", "golden", "hand_example.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line.startswith("A"):
                rows.append([float(v) for v in line.split()[1:]])
            elif line.startswith("case"):
                head, f, S = line[4:].split("|")
                alpha, beta = (float(v) for v in head.split())
                cases.append((alpha, beta,
                              np.array([int(v) for v in f.split()], dtype=np.int32),
                              np.array([int(v) for v in S.split()], dtype=np.int32)))
    return np.array(rows, dtype=np.float32), cases
