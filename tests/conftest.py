import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: test needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(autouse=True)
def _restore_loop_options():
    """Tests that force a mode of the loop kernels (wind_set_loop_options) leave the process-wide default behind them."""
    yield
    from paper_2505_13765_b200 import binding
    if binding._lib is not None:
        binding.wind_set_loop_options()


LOOP_MODES = ["barriers", "counters", "streaming"]


def set_loop_mode(pkg, mode: str) -> None:
    """The three modes of the tensor-core loop: resident weights with grid barriers between the phases, resident weights
    with arrival counters and stamped data (no grid barrier), weights streamed through shared memory every step."""
    if mode == "barriers":
        pkg.wind_set_loop_options(resident=True, dataflow=0)
    elif mode == "counters":
        pkg.wind_set_loop_options(resident=True, dataflow=1)
    elif mode == "streaming":
        pkg.wind_set_loop_options(resident=False)
    else:
        raise ValueError(mode)
