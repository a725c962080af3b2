import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="session")
def trained_tiny_preverify():
    """The pre-verification layer of the tiny pair, trained once per test session on the host with the paper's
    label recipe (a few seconds).  Returns (bf16 tensors for the layer, the training report)."""
    import torch
    from paper_2602_01274_b200 import synth, train_preverify
    torch.set_num_threads(8)
    cfg = synth.CONFIGS["tiny"]
    pair = synth.make_pair(cfg, seed=0, device="cpu", which=("target", "draft"))
    tensors, report = train_preverify.train(cfg, pair, "cpu", n_prompts=128, epochs=10, lr=1e-3, log=lambda *_: None)
    return tensors, report
