"""Structure of the chunk directory (decode step 3) on caches of many small chunks: the check
kernel packs chunks of 16 tiles or fewer side by side in a warp and settles the payload offsets
by comparing every chunk with its predecessor, falling back to the running sum only when that
fails.  Whatever the geometry, a directory whose offsets or lengths were altered (metadata CRC
made right again, so that the structure check is what refuses it) must get the oracle's verdict:
status, first bad chunk and count, where the count follows the running-sum rule (a wrong length
puts every later chunk off, a wrong offset only its own chunk)."""
import struct

import numpy as np
import pytest
import torch

import oracle
from paper_2607_10389_b200 import binding as wm

pytestmark = pytest.mark.gpu
TILE = 16384


def _cache(n, seed):
    rng = np.random.default_rng(seed)
    v = rng.normal(size=(n + 1) // 2).astype(np.float32)
    return (v.view(np.uint32) >> 16).astype("<u2").view(np.uint8)[:n].copy()


def _reseal(w, n, chunk):
    me = oracle.meta_end(n, chunk)
    z = w[:me].copy()
    z[52:56] = 0
    w[52:56] = np.frombuffer(struct.pack("<I", oracle.crc32c(z)), dtype=np.uint8)
    return w


def _verdicts(w, n, chunk, dirty_crc):
    want = oracle.decode_verify(w, n, chunk, dst=np.zeros(n, np.uint8), dst_crc=dirty_crc)[2]
    ws, res = wm.new_workspace(n, chunk), wm.new_result()
    dev = torch.from_numpy(np.concatenate([w, np.zeros((-w.size) % 16, np.uint8)])).cuda()
    dst = torch.zeros(n, dtype=torch.uint8, device="cuda")
    dcrc = torch.from_numpy(dirty_crc.view(np.int32).copy()).cuda()
    wm.wm_decode_verify(dev, w.size, dst, chunk, dcrc, ws, res)
    return wm.read_result(res), want, dst, dcrc


# tiles per chunk: side by side in a warp (1, 2, 3, 5, 16) and one warp per chunk (17, 40)
@pytest.mark.parametrize("tpc,n_chunks", [(1, 70), (2, 37), (3, 45), (5, 13), (16, 5), (17, 4), (40, 3)])
def test_altered_directory_gets_the_oracles_verdict(tpc, n_chunks):
    chunk = tpc * TILE
    n = n_chunks * chunk - (TILE // 2 + 10)            # ragged last tile, short last chunk
    a = _cache(n, 100 + tpc)
    nc = oracle.num_chunks(n, chunk)
    mask = np.ones(nc, np.uint8)
    mask[1::4] = 0                                      # absent chunks in between (their enc_len is 0)
    crc_in = oracle.checksum(a, chunk)
    wire, crc, res = oracle.encode(a, chunk, dirty=mask, crc_in=crc_in)
    # untouched image first: OK on both sides, same bytes
    r, want, dst, dcrc = _verdicts(wire, n, chunk, crc_in.copy())
    assert want.status == 0 and r.ok and np.array_equal(dst.cpu().numpy()[mask.repeat(chunk)[:n] != 0],
                                                         a[mask.repeat(chunk)[:n] != 0])
    rng = np.random.default_rng(tpc)
    seen_counts = set()
    for k in range(24):
        w = wire.copy()
        c = int(rng.integers(0, nc))
        at = 64 + 16 * c
        kind = k % 4
        if kind == 0:                                   # this chunk's offset alone
            po = struct.unpack_from("<Q", w, at)[0]
            struct.pack_into("<Q", w, at, po + 32 * int(rng.integers(1, 9)))
        elif kind == 1:                                 # its length: every later chunk is off the running sum
            el = struct.unpack_from("<I", w, at + 8)[0]
            struct.pack_into("<I", w, at + 8, el + 32)
        elif kind == 2:                                 # a length and the following offsets shifted along: consistent
            el = struct.unpack_from("<I", w, at + 8)[0]                       # neighbours, but the chunk's tiles say otherwise
            struct.pack_into("<I", w, at + 8, el + 64)
            for cc in range(c + 1, nc):
                po = struct.unpack_from("<Q", w, 64 + 16 * cc)[0]
                struct.pack_into("<Q", w, 64 + 16 * cc, po + 64)
        else:                                           # an offset with its high half set
            struct.pack_into("<I", w, at + 4, 1 + int(rng.integers(0, 1 << 20)))
        w = _reseal(w, n, chunk)
        r, want, dst, dcrc = _verdicts(w, n, chunk, crc_in.copy())
        assert want.status_name == "ERR_STRUCT", (tpc, k, want.status_name)
        assert (r.status, r.first_bad_chunk, r.n_bad_chunks) == (want.status, want.first_bad_chunk, want.n_bad_chunks), (tpc, k, c)
        assert np.array_equal(dcrc.cpu().numpy().view(np.uint32), crc_in)
        seen_counts.add(want.n_bad_chunks)
    assert len(seen_counts) >= 3                        # single chunks and long runs of them both occurred


@pytest.mark.parametrize("tpc,nc", [(1, 2100), (3, 1100), (4, 2600)])
def test_many_small_chunks_round_trip_and_mask(tpc, nc):
    """A few tiles per chunk, a few thousand chunks: lists of present chunks, offsets and the
    per-chunk scans at a size where a thread owns several chunks."""
    chunk = tpc * TILE
    n = nc * chunk - 5000
    a = _cache(n, 77)
    rng = np.random.default_rng(5)
    mask = (rng.random(nc) < 0.1).astype(np.uint8)
    mask[-1] = 1
    prev = a.copy()
    for c in np.flatnonzero(mask):
        prev[c * chunk + 17] ^= 0x40
    cur, old = torch.from_numpy(a).cuda(), torch.from_numpy(prev).cuda()
    ws, res = wm.new_workspace(n, chunk), wm.new_result()
    dirty = torch.zeros(nc, dtype=torch.uint8, device="cuda")
    idx = torch.zeros(nc, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    wm.wm_dirty_diff(cur, old, chunk, dirty, idx, cnt, ws)
    assert np.array_equal(dirty.cpu().numpy(), mask) and int(cnt.item()) == int(mask.sum())
    assert np.array_equal(idx.cpu().numpy()[: int(mask.sum())], np.flatnonzero(mask))
    crc_prev = oracle.checksum(prev, chunk)
    want_wire, want_crc, want = oracle.encode(a, chunk, dirty=mask, crc_in=crc_prev)
    crc = torch.from_numpy(crc_prev.view(np.int32).copy()).cuda()
    wire = torch.zeros(wm.wire_bound(n, chunk), dtype=torch.uint8, device="cuda")
    wm.wm_encode(cur, chunk, dirty, crc, wire, ws, res)
    r = wm.read_result(res)
    assert r.ok and r.wire_len == want.wire_len and r.n_present == int(mask.sum())
    assert np.array_equal(wire[: r.wire_len].cpu().numpy(), want_wire)
    assert np.array_equal(crc.cpu().numpy().view(np.uint32), want_crc)
    dcrc = torch.from_numpy(crc_prev.view(np.int32).copy()).cuda()
    wm.wm_decode_verify(wire, r.wire_len, old, chunk, dcrc, ws, res)
    rd = wm.read_result(res)
    assert rd.ok and rd.n_present == int(mask.sum())
    assert torch.equal(old, cur) and np.array_equal(dcrc.cpu().numpy().view(np.uint32), want_crc)
