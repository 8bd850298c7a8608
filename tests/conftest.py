"""pytest configuration: registers the ``gpu`` marker and puts the repo root on sys.path."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
for p in (ROOT, os.path.dirname(os.path.abspath(__file__))):
    if p not in sys.path:
        sys.path.insert(0, p)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu)")


import pytest


@pytest.fixture
def bv_options():
    """Sets tuning / test options of the CUDA library for one test and restores the defaults afterwards."""
    import paper_2403_10444_b200 as bv
    touched = []

    def set_option(name, value):
        touched.append(name)
        bv.bv_set_option(name, value)

    yield set_option
    for name in touched:
        bv.bv_set_option(name, 0)
