import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


_WEIGHTS = {}


def cached_weights(shape, keep=True):
    """(synth.Weights, binding.DeviceWeights) of `shape` with weight seed 0, generated once per test
    session for the shapes several GPU tests share (the 1B-class model, the two-layer variants of
    the 1B- and 7B-class widths).  Host side: bf16 bit patterns, converted on access."""
    import os
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200 import synth
    key = (shape.name, shape.L, shape.d, shape.F, shape.V)
    if key in _WEIGHTS:
        return _WEIGHTS[key]
    W = synth.Weights(shape, 0, cache="bits").prefetch(max(4, min(32, os.cpu_count() or 8)))
    pair = (W, B.DeviceWeights.from_synth(W))
    if keep:
        _WEIGHTS[key] = pair
    return pair
