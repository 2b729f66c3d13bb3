import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def to_oracle_layers(layer_data, rows=None):
    """Widen synthetic tensors (any dtype/device) exactly to fp64 numpy for the checker."""
    from oracle import dp_oracle as O
    out = []
    for ld in layer_data:
        sl = slice(None) if rows is None else rows
        G = ld.G[sl].detach().to("cpu").double().numpy()
        A = None if ld.A is None else ld.A[sl].detach().to("cpu").double().numpy()
        ids = None if ld.ids is None else ld.ids[sl].detach().to("cpu").numpy().astype(np.int64)
        out.append(O.OracleLayer(kind=ld.spec.kind, G=G, A=A, ids=ids, has_bias=ld.spec.has_bias,
                                 vocab=ld.spec.d_in if ld.spec.kind == "embedding" else 0))
    return out


@pytest.fixture
def rng():
    return np.random.default_rng(1234)
