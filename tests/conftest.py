import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(ROOT, "tests", "golden")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


def read_golden(name):
    """Parse a 'key v v v' text fixture into {key: [list of token lists]}."""
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out.setdefault(key, []).append(vals)
    return out


@pytest.fixture(scope="session")
def hand_example():
    import numpy as np
    g = read_golden("hand_example.txt")
    f = lambda rows: np.array([[float(v) for v in r] for r in rows])
    return {
        "m": int(g["m"][0][0]), "n": int(g["n"][0][0]),
        "group": int(g["group"][0][0]), "bits": int(g["bits"][0][0]),
        "W": f(g["W"]).astype(np.float16), "x": f(g["x"])[0].astype(np.float16),
        "t": float(g["t"][0][0]),
        "scales": f(g["scales"]), "zeros": f(g["zeros"]),
        "q": np.array([[int(v) for v in r] for r in g["q"]], dtype=np.uint8),
        "codes": np.array([int(v, 16) for v in g["codes"][0]], dtype=np.uint8),
        "idx": np.array([int(v) for v in g["idx"][0]], dtype=np.int32),
        "y_sparse": f(g["y_sparse"])[0], "y_dense": f(g["y_dense"])[0],
    }
