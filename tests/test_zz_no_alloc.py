"""The allocation-free checksum entry point against the ordinary one.

wm_checksum_noalloc serves callers that cannot allocate device memory when they need a
checksum (under a frozen allocator, in a plug-in that is only handed a stream and buffers, on a
start-up or recovery path that must leave the device heap alone): its scratch and tables are
arrays built into the library.  The test calls it through the C ABI twice in a row on different
inputs, because the built-in scratch is shared by every call and keeps the previous call's
contents, and compares each result with wm_checksum and with the CPU oracle bit for bit
(tolerance 0, as everywhere in this suite).  Two more cases: the call as the very first thing a
fresh process asks of the library (its own set-up path, nothing prepared by another entry point),
and a geometry whose chunks have more tiles than the finishing kernel stages in shared memory.
This file sorts last on purpose: a run that stops at the first failure has then already run every
other test.
"""
import subprocess
import sys
import os
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu
TILE = 16384


def _reference(cache, chunk):
    from paper_2607_10389_b200 import binding as wm
    n = cache.numel()
    ws = wm.new_workspace(n, chunk)
    crc = torch.zeros(wm.num_chunks(n, chunk), dtype=torch.int32, device="cuda")
    wm.wm_checksum(cache, chunk, crc, ws)
    return crc


def test_noalloc_checksum_matches_twice_in_a_row():
    from paper_2607_10389_b200 import binding as wm
    g = torch.Generator(device="cuda").manual_seed(5)
    # two calls back to back: a large ragged cache first, then a smaller one, so that the second
    # call runs over scratch the first one left behind
    for n, chunk in ((37 * TILE * 4 + 5536, 4 * TILE), (9 * TILE + 3, TILE)):
        cache = torch.randint(0, 256, (n,), generator=g, device="cuda", dtype=torch.uint8)
        want = _reference(cache, chunk)
        got = torch.full_like(want, -1)
        wm.wm_checksum_noalloc(cache, chunk, got)
        torch.cuda.synchronize()
        assert torch.equal(got, want), (n, chunk)
        import oracle
        assert np.array_equal(got.cpu().numpy().view(np.uint32), oracle.checksum(cache.cpu().numpy(), chunk)), (n, chunk)
    # and once more on the first geometry: results do not depend on what ran before
    cache = torch.randint(0, 256, (37 * TILE * 4 + 5536,), generator=g, device="cuda", dtype=torch.uint8)
    got = torch.zeros(wm.num_chunks(cache.numel(), 4 * TILE), dtype=torch.int32, device="cuda")
    wm.wm_checksum_noalloc(cache, 4 * TILE, got)
    assert torch.equal(got, _reference(cache, 4 * TILE))


def test_noalloc_checksum_rejects_sizes_beyond_its_scratch():
    from paper_2607_10389_b200 import binding as wm
    cache = torch.zeros(TILE, dtype=torch.uint8, device="cuda")
    crc = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(wm.WmError, match="ERR_ARG"):
        wm.wm_checksum_noalloc(cache, 1 << 20, crc, nbytes=wm.NOALLOC_MAX_BYTES + TILE)
    with pytest.raises(wm.WmError, match="ERR_ARG"):
        wm.wm_checksum_noalloc(cache, 1000, crc)
    wm.wm_checksum_noalloc(cache, TILE, crc)          # still usable after a refusal
    torch.cuda.synchronize()
    assert int(crc.item()) & 0xFFFFFFFF == int(_reference(cache, TILE).item()) & 0xFFFFFFFF


_FIRST_CALL = """
import sys
sys.path.insert(0, {root!r})
import numpy as np, torch
import oracle
from paper_2607_10389_b200 import binding as wm
TILE = 16384
g = torch.Generator(device="cuda").manual_seed(11)
n, chunk = 21 * TILE + 777, 2 * TILE
cache = torch.randint(0, 256, (n,), generator=g, device="cuda", dtype=torch.uint8)
crc = torch.zeros(wm.num_chunks(n, chunk), dtype=torch.int32, device="cuda")
wm.wm_checksum_noalloc(cache, chunk, crc)        # the first call into the library in this process
torch.cuda.synchronize()
assert wm.workspace_status(None) == 0
assert np.array_equal(crc.cpu().numpy().view(np.uint32), oracle.checksum(cache.cpu().numpy(), chunk))
print("first-call ok")
"""


def test_noalloc_checksum_as_the_first_call_of_a_fresh_process():
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-c", _FIRST_CALL.format(root=root)], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "first-call ok" in out.stdout, out.stderr[-2000:]


def test_noalloc_checksum_with_chunks_larger_than_the_finish_stage():
    """Chunks of 8200 tiles (128 MiB and a bit): their digests do not fit the finishing kernel's
    shared-memory stage, so each chunk is folded from global memory; two and a bit chunks."""
    import oracle
    from paper_2607_10389_b200 import binding as wm
    chunk = 8200 * TILE
    n = 2 * chunk + 37 * TILE + 5
    g = torch.Generator(device="cuda").manual_seed(12)
    cache = torch.randint(0, 256, (n,), generator=g, device="cuda", dtype=torch.uint8)
    got = torch.zeros(3, dtype=torch.int32, device="cuda")
    wm.wm_checksum_noalloc(cache, chunk, got)
    torch.cuda.synchronize()
    assert torch.equal(got, _reference(cache, chunk))
    host = cache.cpu().numpy()
    want = [oracle.crc32c(host[c * chunk: (c + 1) * chunk]) for c in range(3)]
    assert got.cpu().numpy().view(np.uint32).tolist() == want
