import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def to_oracle(qt):
    """synth.QuantTensors -> oracle QuantizedMatrix (same arrays, no arithmetic)."""
    from oracle import xfp_oracle as xo
    return xo.QuantizedMatrix(qt.mode, qt.rows, qt.cols, qt.bits, qt.idx, qt.codebook, qt.rowptr, qt.ocol, qt.oval,
                              group_size=qt.group_size, lib_size=qt.lib_size, gid=qt.gid, gscale=qt.gscale,
                              gmid=qt.gmid)


def from_oracle(m):
    """oracle QuantizedMatrix -> synth.QuantTensors (the unpacked input of xfp_pack)."""
    from paper_2605_14844_b200 import synth
    return synth.QuantTensors(m.mode, m.rows, m.cols, m.bits, m.idx, m.codebook, m.rowptr, m.ocol, m.oval,
                              m.group_size, m.lib_size, m.gid, m.gscale, m.gmid)


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


def read_golden(path):
    """Rows of whitespace-separated fields; '#' starts a comment."""
    rows = []
    with open(path) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if line:
                rows.append(line.split())
    return rows
