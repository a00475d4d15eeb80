import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


def pytest_addoption(parser):
    parser.addoption("--full", action="store_true", default=False,
                     help="compare every query row and head of the full-size configurations with the "
                          "oracle instead of a stratified sample (also: UNSTEP_FULL_COMPARE=1)")
