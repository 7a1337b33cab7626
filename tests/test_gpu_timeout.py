"""The give-up paths, run for real: every device-side wait is bounded by time, and when the bound
passes the kernels return, the call reports ERR_TIMEOUT, nothing is installed, nothing is written
out of bounds, and the next call on the same workspace works.

No fault and no hang is involved: the test hook wm_inject_stall leaves out what the waits wait
for (the encode kernel's scanner, the bulk copies of the checksum and decode kernels), and a short
budget (wm_wait_budget_ms) lets the waits run out after a few tens of milliseconds.
"""
import time

import numpy as np
import pytest
import torch

import oracle
from paper_2607_10389_b200 import binding as wm
from paper_2607_10389_b200 import inputs

pytestmark = pytest.mark.gpu

BUDGET_MS = 40


@pytest.fixture
def stalled():
    """Calls issued inside the `with stalled():` block time out; outside it they run normally."""
    class Ctx:
        def __enter__(self):
            wm.wait_budget_ms(BUDGET_MS)
            wm.inject_stall(True)

        def __exit__(self, *a):
            torch.cuda.synchronize()
            wm.inject_stall(False)
            wm.wait_budget_ms(2000)
    yield Ctx
    wm.inject_stall(False)
    wm.wait_budget_ms(2000)


def _cache():
    cfg = inputs.CONFIGS["tiny8m"]
    host = inputs.make_cache(cfg)[: cfg.nbytes - 4321].contiguous()      # ragged tail
    return host, host.cuda(), cfg.chunk_bytes


def test_encode_gives_up_when_no_offset_ever_comes(stalled):
    host, cur, chunk = _cache()
    n = cur.numel()
    nc = wm.num_chunks(n, chunk)
    ws, res = wm.new_workspace(n, chunk), wm.new_result()
    cap = wm.wire_bound(n, chunk)
    wire = torch.full((cap + 4096,), 0xA5, dtype=torch.uint8, device="cuda")
    crc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    t0 = time.time()
    with stalled():
        wm.wm_encode(cur, chunk, None, crc, wire, ws, res, wire_cap=cap)
        r = wm.read_result(res)
    assert r.status_name == "ERR_TIMEOUT"
    assert time.time() - t0 < 20                                     # bounded: the budget, not a hang
    assert wm.workspace_status(ws) == -10
    assert bool((wire[cap:] == 0xA5).all()), "wrote past wire_cap"
    # the same workspace, wire and result record right afterwards, no clean-up in between
    wm.wm_encode(cur, chunk, None, crc, wire, ws, res, wire_cap=cap)
    r = wm.read_result(res)
    want_wire, want_crc, want = oracle.encode(host.numpy(), chunk)
    assert r.ok and r.wire_len == want.wire_len and wm.workspace_status(ws) == 0
    assert np.array_equal(wire[: r.wire_len].cpu().numpy(), want_wire)
    assert np.array_equal(crc.cpu().numpy().view(np.uint32), want_crc)


@pytest.mark.parametrize("options", [0, wm.OPT_ENTROPY, wm.OPT_STRICT])
def test_decode_gives_up_when_the_copies_never_arrive(stalled, options):
    host, cur, chunk = _cache()
    n = cur.numel()
    nc = wm.num_chunks(n, chunk)
    ws, res = wm.new_workspace(n, chunk), wm.new_result()
    wire = torch.zeros(wm.wire_bound(n, chunk), dtype=torch.uint8, device="cuda")
    crc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    wm.wm_encode_opt(cur, chunk, None, crc, wire, ws, res, options & wm.OPT_ENTROPY)
    r = wm.read_result(res)
    assert r.ok
    dst = torch.full((n,), 0x5A, dtype=torch.uint8, device="cuda")
    dst_crc = torch.full((nc,), 7, dtype=torch.int32, device="cuda")
    with stalled():
        wm.wm_decode_verify_opt(wire, r.wire_len, dst, chunk, dst_crc, ws, res, options)
        rd = wm.read_result(res)
    assert rd.status_name == "ERR_TIMEOUT" and wm.workspace_status(ws) == -10
    assert bool((dst_crc == 7).all()), "a checksum was installed after a timeout"
    if options & wm.OPT_STRICT:
        assert bool((dst == 0x5A).all()), "strict decode stored bytes before the verdict"
    wm.wm_decode_verify_opt(wire, r.wire_len, dst, chunk, dst_crc, ws, res, options)
    rd = wm.read_result(res)
    assert rd.ok and torch.equal(dst, cur) and torch.equal(dst_crc, crc)


def test_checksum_calls_fail_closed(stalled):
    host, cur, chunk = _cache()
    n = cur.numel()
    nc = wm.num_chunks(n, chunk)
    ws = wm.new_workspace(n, chunk)
    want = oracle.checksum(host.numpy(), chunk)
    for poly in (None, wm.POLY_ZLIB):
        crc = torch.full((nc,), 0x1234, dtype=torch.int32, device="cuda")
        with stalled():
            if poly is None:
                wm.wm_checksum(cur, chunk, crc, ws)
            else:
                wm.wm_checksum_poly(cur, chunk, poly, crc, ws)
            st = wm.workspace_status(ws)
        assert st == -10 and bool((crc == 0).all()), "digests of data that never arrived were delivered"
    crc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    wm.wm_checksum(cur, chunk, crc, ws)
    assert wm.workspace_status(ws) == 0
    assert np.array_equal(crc.cpu().numpy().view(np.uint32), want)
    # the allocation-free call has the same channel (its built-in scratch: workspace None)
    with stalled():
        crc.fill_(5)
        wm.wm_checksum_noalloc(cur, chunk, crc)
        st = wm.workspace_status(None)
    assert st == -10 and bool((crc == 0).all())
    wm.wm_checksum_noalloc(cur, chunk, crc)
    assert wm.workspace_status(None) == 0
    assert np.array_equal(crc.cpu().numpy().view(np.uint32), want)


def test_dirty_diff_leaves_a_clean_status_even_on_a_dirty_workspace(stalled):
    host, cur, chunk = _cache()
    n = cur.numel()
    nc = wm.num_chunks(n, chunk)
    ws = wm.new_workspace(n, chunk)
    crc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    with stalled():
        wm.wm_checksum(cur, chunk, crc, ws)
        assert wm.workspace_status(ws) == -10
    prev = cur.clone()
    prev[chunk * 3 + 17] ^= 1
    dirty = torch.zeros(nc, dtype=torch.uint8, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    wm.wm_dirty_diff(cur, prev, chunk, dirty, None, cnt, ws)         # no waits inside: cannot time out
    assert wm.workspace_status(ws) == 0 and int(cnt.item()) == 1 and int(dirty[3].item()) == 1
