"""The calls allocate nothing and never synchronise, so a whole step (checksum, dirty diff, encode,
decode + verify: 13 kernels with their programmatic-launch edges) can be captured in a CUDA graph
and replayed; the replay must produce what the eager calls produce."""
import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu
TILE = 16384


@pytest.mark.parametrize("entropy", [False, True])
def test_a_captured_step_replays_bit_for_bit(entropy):
    import torch
    from paper_2607_10389_b200 import binding as wm
    rng = np.random.default_rng(3)
    n, chunk = 23 * TILE + 999, 4 * TILE
    a = (rng.normal(size=(n + 1) // 2).astype(np.float32).view(np.uint32) >> 16).astype("<u2").view(np.uint8)[:n].copy()
    b = a.copy()
    b[5 * TILE + 3] ^= 1
    b[19 * TILE:] = 0
    opt = wm.OPT_ENTROPY if entropy else 0
    nc = wm.num_chunks(n, chunk)
    cur, prev = torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()
    ws = wm.new_workspace(n, chunk)
    wire = torch.zeros(wm.wire_bound(n, chunk), dtype=torch.uint8, device="cuda")
    shadow = torch.zeros(n, dtype=torch.uint8, device="cuda")
    crc, crc_e, crc_d = (torch.zeros(nc, dtype=torch.int32, device="cuda") for _ in range(3))
    dirty = torch.zeros(nc, dtype=torch.uint8, device="cuda")
    idx = torch.zeros(nc, dtype=torch.int32, device="cuda")
    nd = torch.zeros(1, dtype=torch.int32, device="cuda")
    res_e, res_d = wm.new_result(), wm.new_result()
    want_wire, want_crc, want_res = oracle.encode(a, chunk, entropy=entropy)
    want_dirty, want_idx = oracle.dirty_diff(a, b, chunk)

    def step(stream):
        wm.wm_checksum(cur, chunk, crc, ws, stream=stream)
        wm.wm_dirty_diff(cur, prev, chunk, dirty, idx, nd, ws, stream=stream)
        wm.wm_encode_opt(cur, chunk, None, crc_e, wire, ws, res_e, opt, stream=stream)
        wm.wm_decode_verify_opt(wire, want_res.wire_len, shadow, chunk, crc_d, ws, res_d, opt, stream=stream)

    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        step(s)                                     # first use sets the library up: before any capture
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            step(torch.cuda.current_stream())
    for t in (wire, shadow, crc, crc_e, crc_d, dirty, idx, nd):
        t.zero_()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    re_, rd = wm.read_result(res_e), wm.read_result(res_d)
    assert re_.ok and rd.ok and re_.wire_len == want_res.wire_len
    assert np.array_equal(wire[: re_.wire_len].cpu().numpy(), want_wire)
    assert np.array_equal(shadow.cpu().numpy(), a)
    for c in (crc, crc_e, crc_d):
        assert np.array_equal(c.cpu().numpy().view(np.uint32), want_crc)
    assert np.array_equal(dirty.cpu().numpy(), want_dirty) and int(nd.item()) == len(want_idx)
    # new data in the same buffers: the replay works on what is there now (the previous snapshot
    # catches up, so no chunk is dirty any more; the image length, a host argument frozen into
    # the captured decode call, stays what it was because the cache did)
    prev.copy_(cur)
    shadow.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert wm.read_result(res_d).ok and np.array_equal(shadow.cpu().numpy(), a) and int(nd.item()) == 0
    assert not bool(dirty.any())
