import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); skipped by -m 'not gpu'")


@pytest.fixture(scope="session")
def c1_inputs():
    from paper_2609_29812_b200 import workloads
    return workloads.make_layer_inputs(workloads.config1(), seed=0)


def pytest_sessionfinish(session, exitstatus):
    """FL_PARITY_LOG=<path>: write the measured error of every attention comparison (relative L2, max abs) there."""
    path = os.environ.get("FL_PARITY_LOG")
    if not path:
        return
    import json
    import helpers
    worst = {}
    for what, carried, rel, mx, bound in helpers.ERROR_LOG:
        key = (what.split(" h")[0] if " h" in what else what, carried)
        w = worst.setdefault(key, [0.0, 0.0, 0, 0.0])
        w[0], w[1], w[2], w[3] = max(w[0], rel), max(w[1], mx), w[2] + 1, max(w[3], bound)
    with open(path, "w") as f:
        for (what, carried), (rel, mx, n, bound) in sorted(worst.items()):
            f.write(json.dumps({"check": what, "carried_roundings": carried, "comparisons": n, "max_rel_l2": rel,
                                "max_abs": mx, "max_abs_bound": bound}) + "\n")
