import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def oracle_lib():
    from oracle.hap_oracle import build_oracle
    return build_oracle()


def pytest_sessionfinish(session, exitstatus):
    """When the suite runs on the self-checking build (HAP_LIBRARY=checked), no check site may have fired."""
    if os.environ.get("HAP_LIBRARY") != "checked":
        return
    try:
        import torch
        if not torch.cuda.is_available():
            return
        import paper_2609_39350_b200 as hap
        sites = hap.hap_self_check()
    except Exception as e:                      # the library was never loaded in this session
        print(f"\nself-check word not read: {e}")
        return
    if sites:
        print(f"\nself-checking build: check sites fired: {sites:#x}")
        session.exitstatus = 1
    else:
        print("\nself-checking build: no check site fired")
