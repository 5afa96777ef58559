import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def load_hand_examples():
    """Parse tests/golden/quantizer_hand_examples.txt into a list of dicts."""
    path = os.path.join(ROOT, "tests", "golden", "quantizer_hand_examples.txt")
    out, cur = [], None
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] == "bits":
            cur = dict(bits=int(tok[1]), lo=float(tok[3]), hi=float(tok[5]))
            out.append(cur)
        elif tok[0] == "x":
            cur["x"] = [float(t) for t in tok[1:]]
        elif tok[0] == "codes":
            cur["codes"] = [int(t) for t in tok[1:]]
        elif tok[0] == "bytes":
            cur["bytes"] = bytes(int(t, 16) for t in tok[1:])
    return out


@pytest.fixture(scope="session")
def hand_examples():
    return load_hand_examples()


_INDEX_CHECK_REPORT = []


def pytest_terminal_summary(terminalreporter):
    for line in _INDEX_CHECK_REPORT:
        terminalreporter.write_line(line)


@pytest.fixture(scope="session", autouse=True)
def index_checked_build_reports_clean(request):
    """When the tests run against the library built with index checks (QUANTPIPE_LIB points at it), the
    session ends by reading the status once more: no index may have been out of range."""
    yield
    if not os.environ.get("QUANTPIPE_LIB"):
        return
    import torch
    if not torch.cuda.is_available():
        return
    import paper_2211_04515_b200 as qp
    assert qp.qp_built_with_index_checks()
    c = qp.Context(0)
    assert c.qp_get_status() & qp.QP_DEV_INDEX_RANGE == 0
    c.close()
    _INDEX_CHECK_REPORT.append("index checks: on, no index out of range")
