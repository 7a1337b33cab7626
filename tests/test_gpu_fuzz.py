"""Seeded random geometries, masks, data recipes and codec options: the GPU's wire image, checksums
and result record against the oracle's, then the round trip.  Tolerance 0."""
import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu
TILE = 16384


def _data(rng, n):
    kind = rng.integers(0, 5)
    if kind == 0:                                             # Gaussian at a random scale
        v = (rng.normal(size=(n + 1) // 2) * float(2.0 ** rng.integers(-30, 30))).astype(np.float32)
        a = (v.view(np.uint32) >> 16).astype("<u2").view(np.uint8)[:n].copy()
    elif kind == 1:                                           # random bytes (raw tiles, NaN and Inf patterns)
        a = rng.integers(0, 256, n, dtype=np.uint8)
    elif kind == 2:                                           # per-tile mixture, some tiles zero or constant
        a = np.empty(n, dtype=np.uint8)
        for o in range(0, n, TILE):
            m = min(TILE, n - o)
            k = rng.integers(0, 4)
            if k == 0:
                a[o:o + m] = 0
            elif k == 1:
                a[o:o + m] = np.resize(np.array([0x80, 0x3F], dtype=np.uint8), m)
            elif k == 2:
                a[o:o + m] = rng.integers(0, 256, m, dtype=np.uint8)
            else:
                v = (rng.normal(size=(m + 1) // 2) * 3.0).astype(np.float32)
                a[o:o + m] = (v.view(np.uint32) >> 16).astype("<u2").view(np.uint8)[:m]
    elif kind == 3:                                           # wide exponent spread inside groups
        e = rng.integers(0, 256, (n + 1) // 2).astype(np.uint32)
        m = rng.integers(0, 128, (n + 1) // 2).astype(np.uint32)
        s = rng.integers(0, 2, (n + 1) // 2).astype(np.uint32)
        a = ((s << 15) | (e << 7) | m).astype("<u2").view(np.uint8)[:n].copy()
    else:                                                     # narrow exponent spread: widths 0..3
        e = (100 + rng.integers(0, int(rng.integers(1, 9)), (n + 1) // 2)).astype(np.uint32)
        m = rng.integers(0, 128, (n + 1) // 2).astype(np.uint32)
        a = ((e << 7) | m).astype("<u2").view(np.uint8)[:n].copy()
    return a


@pytest.mark.parametrize("seed", range(48))
def test_random_case_matches_the_oracle(seed):
    import torch
    from paper_2607_10389_b200 import binding as wm
    rng = np.random.default_rng(1000 + seed)
    chunk = int(rng.choice([1, 2, 3, 4, 8])) * TILE
    n = int(rng.integers(1, 40 * TILE))
    if rng.integers(0, 4) == 0:
        n = max(TILE, n // TILE * TILE)                       # no ragged tail
    option = ["default", "zero", "entropy", "zero+entropy"][seed % 4]
    a = _data(rng, n)
    nc = oracle.num_chunks(n, chunk)
    masked = bool(rng.integers(0, 2))
    dirty = (rng.integers(0, 3, nc) > 0).astype(np.uint8) if masked else None
    crc_in = oracle.checksum(a, chunk)
    stale = crc_in.copy()
    want, want_crc, want_res = oracle.encode(a, chunk, dirty=dirty, crc_in=stale, zero_tiles="zero" in option,
                                             entropy="entropy" in option)
    wm.zero_tiles_enable("zero" in option)
    wm.entropy_enable("entropy" in option)
    try:
        ws = wm.new_workspace(n, chunk)
        wire = torch.full((wm.wire_bound(n, chunk),), 0xC3, dtype=torch.uint8, device="cuda")
        crc = torch.from_numpy(stale.view(np.int32).copy()).cuda()
        res = wm.new_result()
        d = None if dirty is None else torch.from_numpy(dirty).cuda()
        wm.wm_encode(torch.from_numpy(a).cuda(), chunk, d, crc, wire, ws, res)
        r = wm.read_result(res)
        assert (r.status, r.wire_len, r.payload_bytes, r.n_present, r.cache_crc) == (
            want_res.status, want_res.wire_len, want_res.payload_bytes, want_res.n_present, want_res.cache_crc)
        assert np.array_equal(wire[: r.wire_len].cpu().numpy(), want)
        assert np.array_equal(crc.cpu().numpy().view(np.uint32), want_crc)
        # decode over a destination that holds the absent chunks already
        base = a.copy()
        if dirty is not None:
            for c in range(nc):
                if dirty[c]:
                    base[c * chunk:(c + 1) * chunk] = 0x77
        dst = torch.from_numpy(base).cuda()
        dcrc = torch.from_numpy(stale.view(np.int32).copy()).cuda()
        strict = bool(rng.integers(0, 2))
        (wm.wm_decode_verify_strict if strict else wm.wm_decode_verify)(wire, r.wire_len, dst, chunk, dcrc, ws, res)
        rd = wm.read_result(res)
        assert rd.status == 0 and np.array_equal(dst.cpu().numpy(), a)
        assert np.array_equal(dcrc.cpu().numpy().view(np.uint32), want_crc)
    finally:
        wm.zero_tiles_enable(False)
        wm.entropy_enable(False)


@pytest.mark.parametrize("seed", range(32))
def test_random_leaf_tables_match_the_flat_image(seed):
    """The cache cut into leaves at random places (tile boundaries, 16-, 4-, 2-byte and odd
    offsets, runs of tiny leaves), every option set, with and without a mask: the image is the
    oracle's image of the concatenation and the decode lands in a second, differently cut set of
    leaves."""
    import torch
    from paper_2607_10389_b200 import binding as wm
    rng = np.random.default_rng(3000 + seed)
    chunk = int(rng.choice([1, 2, 4])) * TILE
    nt = int(rng.integers(3, 48))
    n = nt * TILE + int(rng.integers(0, 2)) * int(rng.integers(1, TILE))
    a = _data(rng, n)
    opt = seed % 4
    nc = oracle.num_chunks(n, chunk)
    dirty = (rng.integers(0, 3, nc) > 0).astype(np.uint8) if seed % 2 else None
    stale = oracle.checksum(a, chunk)
    want, want_crc, want_res = oracle.encode(a, chunk, dirty=dirty, crc_in=stale, zero_tiles=bool(opt & 1), entropy=bool(opt & 2))

    def cut(k):
        # granularity of the cut positions: whole tiles (as an engine's large tensors), or any
        # multiple of 16 / 4 / 2 / 1 bytes; now and then a run of tiny leaves (scalar flags)
        gran = int(rng.choice([TILE, 16, 4, 2, 1]))
        edges = set(int(x) * gran for x in rng.integers(1, max(2, n // gran), k))
        if rng.integers(0, 2):
            o = int(rng.integers(1, n - 200))
            for size in rng.choice([1, 2, 4, 8, 64], int(rng.integers(1, 12))):
                o += int(size)
                edges.add(o)
        bounds = [0] + sorted(e for e in edges if 0 < e < n) + [n]
        return [(bounds[i], bounds[i + 1]) for i in range(len(bounds) - 1) if bounds[i + 1] > bounds[i]]

    src = [torch.from_numpy(a[lo:hi].copy()).cuda() for lo, hi in cut(int(rng.integers(1, 9)))]
    ws = wm.new_workspace(n, chunk)
    wire = torch.full((wm.wire_bound(n, chunk),), 0x3C, dtype=torch.uint8, device="cuda")
    crc = torch.from_numpy(stale.view(np.int32).copy()).cuda()
    res = wm.new_result()
    d = None if dirty is None else torch.from_numpy(dirty).cuda()
    wm.wm_encode_opt(None, chunk, d, crc, wire, ws, res, opt, leaf_table=wm.make_leaf_table(src), nbytes=n)
    r = wm.read_result(res)
    assert r.status == 0 and r.wire_len == want_res.wire_len
    assert np.array_equal(wire[: r.wire_len].cpu().numpy(), want) and np.array_equal(crc.cpu().numpy().view(np.uint32), want_crc)
    base = a.copy()
    if dirty is not None:
        for c in range(nc):
            if dirty[c]:
                base[c * chunk:(c + 1) * chunk] = 0x77
    spans = cut(int(rng.integers(1, 9)))
    dst = [torch.from_numpy(base[lo:hi].copy()).cuda() for lo, hi in spans]
    dcrc = torch.from_numpy(stale.view(np.int32).copy()).cuda()
    wm.wm_decode_verify_opt(wire, r.wire_len, None, chunk, dcrc, ws, res, (opt & 2) | (wm.OPT_STRICT if seed % 3 == 0 else 0),
                            leaf_table=wm.make_leaf_table(dst), nbytes=n)
    assert wm.read_result(res).status == 0
    for (lo, hi), t in zip(spans, dst):
        assert np.array_equal(t.cpu().numpy(), a[lo:hi])


@pytest.mark.parametrize("seed", range(12))
def test_buffers_at_odd_sixteen_byte_offsets(seed):
    """The ABI asks for 16-byte alignment and nothing more: cache, previous snapshot, wire image,
    destination and workspace each start 16, 48, 80 ... bytes into their allocations."""
    import torch
    from paper_2607_10389_b200 import binding as wm
    rng = np.random.default_rng(4000 + seed)
    chunk = int(rng.choice([1, 2, 4])) * TILE
    n = int(rng.integers(1, 30 * TILE))
    a = _data(rng, n)
    b = a.copy()
    for _ in range(int(rng.integers(0, 4))):
        b[int(rng.integers(0, n))] ^= 0x10
    opt = seed % 4
    nc = oracle.num_chunks(n, chunk)

    def at_offset(nbytes, fill=None):
        off = 16 * int(rng.integers(1, 16)) | 16
        t = torch.empty(nbytes + off + 64, dtype=torch.uint8, device="cuda")
        v = t[off: off + nbytes]
        assert v.data_ptr() % 16 == 0 and v.data_ptr() % 32 != 0
        if fill is not None:
            v.copy_(torch.from_numpy(fill))
        return v

    cur, prev = at_offset(n, a), at_offset(n, b)
    ws = at_offset(wm.workspace_bytes(n, chunk))
    wire = at_offset(wm.wire_bound(n, chunk))
    dst = at_offset(n)
    crc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    res = wm.new_result()
    wm.wm_checksum(cur, chunk, crc, ws)
    assert np.array_equal(crc.cpu().numpy().view(np.uint32), oracle.checksum(a, chunk))
    dirty = torch.zeros(nc, dtype=torch.uint8, device="cuda")
    idx = torch.zeros(nc, dtype=torch.int32, device="cuda")
    nd = torch.zeros(1, dtype=torch.int32, device="cuda")
    wm.wm_dirty_diff(cur, prev, chunk, dirty, idx, nd, ws)
    want_dirty, want_idx = oracle.dirty_diff(a, b, chunk)
    assert np.array_equal(dirty.cpu().numpy(), want_dirty) and int(nd.item()) == len(want_idx)
    want, want_crc, want_res = oracle.encode(a, chunk, zero_tiles=bool(opt & 1), entropy=bool(opt & 2))
    wm.wm_encode_opt(cur, chunk, None, crc, wire, ws, res, opt)
    r = wm.read_result(res)
    assert r.status == 0 and np.array_equal(wire[: r.wire_len].cpu().numpy(), want)
    dcrc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    wm.wm_decode_verify_opt(wire, r.wire_len, dst, chunk, dcrc, ws, res, opt & 2)
    assert wm.read_result(res).status == 0 and np.array_equal(dst.cpu().numpy(), a)
    h = torch.zeros(nc, dtype=torch.int64, device="cuda")
    wm.wm_checksum_xxh64(cur, chunk, seed, h)
    assert np.array_equal(h.cpu().numpy().view(np.uint64), oracle.checksum_xxh64(a, chunk, seed))
