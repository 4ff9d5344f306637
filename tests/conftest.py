import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200, sm_100a)")


def read_layer_map_golden():
    rows = []
    with open(os.path.join(ROOT, "tests", "golden", "layer_maps.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            kind, name, nb, na, ret, jm = [s.strip() for s in line.split("|")]
            rows.append(dict(kind=kind, name=name, n_base=int(nb), n_aux=int(na),
                             retained=None if ret == "-" else [int(x) for x in ret.split()],
                             map=[int(x) for x in jm.split()]))
    return rows
