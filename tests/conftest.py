import os
import sys

import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def pytest_collection_modifyitems(config, items):
    import torch
    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_sessionfinish(session, exitstatus):
    """When the session ran on the checking build of the library (MOE_B200_LIB points at it), no kernel may have
    seen an index outside its range: the count is part of the result."""
    if not os.environ.get("MOE_B200_LIB"):
        return
    from paper_1701_06538_b200 import binding as B
    if B._lib is None:
        return
    seen = B.moe_debug_bounds_violations()
    expect = int(os.environ.get("MOE_EXPECT_VIOLATIONS", "0"))
    print(f"\nchecking build: {seen} out-of-range indices seen (expected {'some' if expect else 'none'})")
    if (seen != 0) != bool(expect):
        session.exitstatus = 1
