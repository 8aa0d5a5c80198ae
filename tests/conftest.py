import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200, sm_100a)")


@pytest.fixture(scope="session")
def oracle():
    from oracle import jv_oracle
    jv_oracle.build()
    return jv_oracle


def pytest_sessionfinish(session, exitstatus):
    """Every bf16 parity comparison of the session (plain metric, metric with the store-rounding
    allowance, bf16 store floor of the oracle output) as one JSON line each, where a run keeps its
    artefacts."""
    import json
    from tests import _util
    out = os.path.join(ROOT, "gpurun_out")
    if _util.PARITY_LOG and os.path.isdir(out):
        with open(os.path.join(out, "parity_metrics.jsonl"), "w") as f:
            for rec in _util.PARITY_LOG:
                f.write(json.dumps(rec) + "\n")
