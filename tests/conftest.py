import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs on a B200 box)")


def load_golden_vectors():
    path = os.path.join(ROOT, "tests", "golden", "quantizer_vectors.txt")
    cases, cur = [], None
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, *vals = line.split()
        if key == "case":
            cur = {"name": vals[0]}
            cases.append(cur)
        elif key == "bits":
            cur["bits"] = int(vals[0])
        elif key in ("d", "qhat"):
            cur[key] = [float(v) for v in vals]
        elif key == "k":
            cur["k"] = [int(v) for v in vals]
        elif key == "scale":
            cur["scale"] = float(vals[0])
        elif key == "bytes":
            cur["bytes"] = bytes(int(v, 16) for v in vals)
    return cases


@pytest.fixture(scope="session")
def golden_vectors():
    return load_golden_vectors()
