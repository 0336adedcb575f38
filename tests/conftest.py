import os
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def pytest_collection_modifyitems(config, items):
    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def dense_rows(kv, tensor, layer, b, h, positions):
    """Rows of one (layer, sequence, KV head) at the given positions, as fp64 [n, D].

    Index arithmetic restated here on purpose (page -> physical page -> row) so that the
    tests do not lean on either implementation's addressing code.
    """
    flat = tensor.reshape(-1)
    rows = []
    for pos in positions:
        page, slot = divmod(int(pos), kv.page_size)
        phys = kv.phys_page(b, page)
        off = (layer * kv.layer_stride + phys * kv.page_stride + h * kv.head_stride
               + slot * kv.slot_stride)
        rows.append(flat[off:off + kv.head_dim])
    return torch.stack(rows).to(torch.float64)
