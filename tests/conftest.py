import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


def load_hand_examples():
    path = os.path.join(ROOT, "tests", "golden", "hand_examples.txt")
    out = []
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        name, rows, rng, sm = [s.strip() for s in line.split(";")]
        M = [[int(x) for x in r.split()] for r in rows.split("|")]

        def parse(s):
            w, b, idx = s.split(",")
            return int(w), int(b), [int(x) for x in idx.split()]
        out.append((name, M, parse(rng), parse(sm)))
    return out


@pytest.fixture(scope="session")
def hand_examples():
    return load_hand_examples()
