import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200, sm_100a)")


def pytest_sessionfinish(session, exitstatus):
    """With CAFEQ_TIE_LOG=<file>, write the fraction of codes that differed from the oracle inside the tie window,
    one line per tie-aware comparison of the run."""
    path = os.environ.get("CAFEQ_TIE_LOG")
    if not path:
        return
    try:
        sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
        import parity_utils
        with open(path, "w") as f:
            for label, frac, n in parity_utils.TIE_FRACTIONS:
                f.write(f"{label}\t{n}\t{frac:.3e}\n")
    except Exception as exc:  # a log, never a failure
        print("tie log not written:", exc)
