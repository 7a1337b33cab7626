"""The C-ABI library loads without a GPU and exports every function include/wm.h declares;
geometry helpers (pure host arithmetic) agree with the oracle's."""
import ctypes
import os
import re

import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "wm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(wm_[a-z0-9_]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    from paper_2607_10389_b200 import build
    return ctypes.CDLL(build.build())


def test_every_declared_function_is_exported(lib):
    names = _declared()
    assert {"wm_checksum", "wm_dirty_diff", "wm_encode", "wm_decode_verify"} <= set(names)
    for n in names:
        assert getattr(lib, n) is not None, n


def test_binding_lists_the_same_entry_points():
    from paper_2607_10389_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_geometry_helpers_match_oracle():
    from paper_2607_10389_b200 import binding as wm
    for n, chunk in ((1, 16384), (16384, 16384), (1_670_124_960, 4 << 20), (1_671_168_000, 1 << 20),
                     (1 << 30, 1 << 20), (17_179_869_184, 4 << 20), (148456, 65536)):
        assert wm.num_chunks(n, chunk) == oracle.num_chunks(n, chunk)
        assert wm.num_tiles(n) == oracle.num_tiles(n)
        assert wm.meta_bytes(n, chunk) == oracle.meta_end(n, chunk)
        assert wm.wire_bound(n, chunk) == oracle.wire_bound(n, chunk)
        assert wm.workspace_bytes(n, chunk) > 12 * wm.num_tiles(n)
    assert wm.workspace_bytes(100, 1000) == 0 and wm.workspace_bytes(0, 16384) == 0


def test_calls_refuse_to_run_without_a_device_or_on_host_tensors():
    import torch
    from paper_2607_10389_b200 import binding as wm
    a = torch.zeros(16384, dtype=torch.uint8)
    with pytest.raises(wm.WmError):
        wm.wm_checksum(a, 16384, torch.zeros(1, dtype=torch.int32), torch.zeros(1024, dtype=torch.uint8))
