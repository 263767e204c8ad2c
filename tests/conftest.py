import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


@pytest.fixture(scope="session")
def c0():
    """Tiny workload: weights, prefix, oracle (float64)."""
    from synth_inputs import configs as C, data
    from oracle.specvla import SpecVLAOracle
    w = data.make_weights(C.TINY, C.C0.seed)
    embeds, ids = data.make_prefix(C.C0)
    return dict(wl=C.C0, desc=C.TINY, weights=w, embeds=embeds, ids=ids,
                make=lambda **kw: SpecVLAOracle(C.TINY, w, **kw))
