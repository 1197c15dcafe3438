import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


@pytest.fixture(scope="session")
def tiny_inputs():
    """Weights, frequency tables and prefix of the tiny workload (built once per session, on the CPU)."""
    import spd_inputs as si

    wl = si.get_workload("tiny")
    weights = si.make_weights(wl.shape, seed=0)
    tables = si.make_ngram_tables(wl.shape.vocab, wl.zipf_s, wl.stream_len, wl.orders, wl.retain, seed=1)
    prefix = si.make_prefix(wl.prefix_kind, wl.prefix_len, wl.shape.vocab, wl.zipf_s, seed=2)
    return wl, weights, tables, prefix
