import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def pytest_terminal_summary(terminalreporter):
    """Largest errors of the fused calls against the oracle's fp64 results, as measured in this run."""
    import helpers

    if helpers.FUSED_MAXIMA:
        terminalreporter.write_line("fused calls, largest error seen: |y - ref| / sum|w x|, plain relative (|ref| >= 0.1 rms)")
        for label, (scaled, plain) in sorted(helpers.FUSED_MAXIMA.items()):
            terminalreporter.write_line(f"  {label:24s} {scaled:.3e}  {plain:.3e}")


@pytest.fixture(scope="session")
def eo():
    from oracle import ecco_oracle

    ecco_oracle.lib()
    return ecco_oracle


@pytest.fixture(scope="session")
def synth():
    from paper_2505_06901_b200 import synth as s

    return s


@pytest.fixture(scope="session")
def cfg1_small(eo, synth):
    """Config-1 distribution at reduced size: metadata calibrated by the oracle on 2048 groups of
    a separate seeded matrix, and a 256x1024 weight slice (2048 groups) to encode."""
    cal = synth.weight_matrix(256, 1024, 2001)
    w = synth.weight_matrix(256, 1024, 1001)
    meta = eo.calibrate(cal, S=64, H=4, seed=1, select=eo.SELECT_MSE)
    eo.set_exponent(meta, w)
    blocks, stats = eo.encode(meta, w, eo.SELECT_MSE)
    return dict(meta=meta, w=w, cal=cal, blocks=blocks, stats=stats)


@pytest.fixture(scope="session")
def kv_small(eo, synth):
    """Config-3 distribution at reduced size: K cache [2][4][256][128], min/max pattern selection."""
    cal = synth.kv_cache(2, 4, 256, 2003, 3003)
    k = synth.kv_cache(2, 4, 256, 1003, 3003)
    meta = eo.calibrate(cal, S=64, H=4, seed=3, select=eo.SELECT_MINMAX)
    blocks, stats = eo.encode(meta, k, eo.SELECT_MINMAX)
    return dict(meta=meta, k=k, cal=cal, blocks=blocks, stats=stats)
