import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def pytest_collection_modifyitems(config, items):
    import torch

    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(autouse=True)
def guard(request, monkeypatch):
    """GPU tests: every workspace the binding or a test allocates through chai.new_workspace gets guard bands,
    verified when the test ends; `guard.empty_like(x)` gives a test the same for its outputs."""
    if "gpu" not in request.keywords:
        yield None
        return
    import torch
    if not torch.cuda.is_available():
        yield None
        return
    from guard import Guards
    from paper_2403_08058_b200 import chai
    g = Guards("cuda")
    monkeypatch.setattr(chai, "new_workspace", g.workspace)
    yield g
    g.check()
