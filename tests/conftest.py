import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


# AASD_SEED_OFFSET=n adds n to every integer seed the tests hand to numpy: the same suite on
# other draws (a soak run), without touching a test.  Unset or 0: the committed seeds.
_SEED_OFFSET = int(os.environ.get("AASD_SEED_OFFSET", "0") or 0)
if _SEED_OFFSET:
    import numpy as _np

    _default_rng = _np.random.default_rng

    def _shifted_rng(seed=None):
        if isinstance(seed, (int, _np.integer)):
            seed = int(seed) + _SEED_OFFSET
        return _default_rng(seed)

    _np.random.default_rng = _shifted_rng
