import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_addoption(parser):
    parser.addoption("--sl-debug-bounds", action="store_true", default=False,
                     help="run the tests against the bounds-checked debug build of the library "
                          "(csrc/libsparseloco_debug.so) instead of the normal one")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")
    if config.getoption("--sl-debug-bounds"):
        from paper_2601_02360_b200 import build
        build.LIB_PATH = build.build(debug=True)      # the binding loads whatever LIB_PATH names
