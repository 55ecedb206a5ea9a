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


# ---------------------------------------------------------------------------------------------------------
# Guard words.  Every output tensor the package allocates goes through api._new; in the GPU tests that function is
# replaced by one that surrounds the tensor with a known pattern, and after each test the patterns are checked: a
# kernel that writes before or behind one of its outputs fails the test that ran it.
# ---------------------------------------------------------------------------------------------------------
GUARD_BYTES = 512
GUARD_BYTE = 0xA5


@pytest.fixture(autouse=True)
def guard_words(request, monkeypatch):
    if "gpu" not in request.keywords:
        yield
        return
    import torch
    from paper_2402_14160_b200 import api
    made = []

    def guarded_new(shape, dtype, device):
        shape = tuple(int(x) for x in (shape if isinstance(shape, (tuple, list, torch.Size)) else (shape,)))
        n = 1
        for x in shape:
            n *= x
        item = torch.empty((), dtype=dtype).element_size()
        pad = (-n * item) % 256                                  # keeps the tensor itself 256-byte aligned
        raw = torch.full((GUARD_BYTES + n * item + pad + GUARD_BYTES,), GUARD_BYTE, dtype=torch.uint8, device=device)
        made.append((raw, n * item))
        return raw[GUARD_BYTES:GUARD_BYTES + n * item].view(dtype).view(shape)

    monkeypatch.setattr(api, "_new", guarded_new)
    yield
    if made:
        torch.cuda.synchronize()
        for raw, nbytes in made:
            front, back = raw[:GUARD_BYTES], raw[GUARD_BYTES + nbytes:]
            assert bool((front == GUARD_BYTE).all()) and bool((back == GUARD_BYTE).all()), \
                "a kernel wrote outside an output tensor of %d bytes" % nbytes
