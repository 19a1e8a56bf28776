import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a); run with -m gpu")


def pytest_collection_modifyitems(config, items):
    # GPU tests never run silently on a machine without a GPU.
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="module", autouse=True)
def _library_options_are_process_wide():
    """The library's options are process-wide, so a test module that leaves one changed would
    silently change every later module.  After each module: every option must be back at its
    documented default (the assertion names the module's leak), and is put back regardless."""
    yield
    from paper_2603_24517_b200 import binding
    if binding._lib is None:   # the module never loaded the library
        return
    left = {n: binding.attn_get_option(n) for n in binding.OPTION_DEFAULTS}
    for n, d in binding.OPTION_DEFAULTS.items():
        binding.attn_set_option(n, d)
    assert left == binding.OPTION_DEFAULTS, f"options left changed by this module: {left}"
