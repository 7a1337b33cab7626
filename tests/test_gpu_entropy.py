"""ENT tiles on the GPU (wm_entropy_enable) against the oracle: wire images bit for bit, decoded
caches, checksums and verdicts on damaged images."""
import struct

import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu
TILE = 16384


@pytest.fixture()
def wm():
    from paper_2607_10389_b200 import binding
    binding.entropy_enable(True)
    yield binding
    binding.entropy_enable(False)


def _gauss(n_elems, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    return ((rng.normal(size=n_elems) * scale).astype(np.float32).view(np.uint32) >> 16).astype("<u2")


def _mixed_cache(n, seed):
    """Gaussian data at several scales, a tile of random bytes (stays raw), special values, a tile
    with one wild strand (escapes), a constant tile."""
    rng = np.random.default_rng(seed)
    v = _gauss((n + 1) // 2, seed)
    a = v.view(np.uint8)[:n].copy()
    nt = n // TILE
    if nt >= 2:
        a[TILE:2 * TILE] = rng.integers(0, 256, TILE, dtype=np.uint8)
    if nt >= 3:
        t = a[2 * TILE:3 * TILE].view("<u2")
        t[:] = _gauss(8192, seed + 1, 300.0)
        t[:6] = [0x7FC0, 0xFF80, 0x0001, 0x8000, 0x7F80, 0x0000]
    if nt >= 4:
        t = a[3 * TILE:4 * TILE].view("<u2")
        t[:] = 0x3F80
        t[0::64] = rng.integers(0, 65536, 128).astype("<u2")       # word 0 of every row: strand 0 of every share
    if nt >= 5:
        a[4 * TILE:5 * TILE].view("<u2")[:] = 0xC2F7
    if nt >= 6:
        a[5 * TILE:6 * TILE].view("<u2")[:] = _gauss(8192, seed + 2, 1e-20)
    return a


def _run_encode(wm, a, chunk, dirty=None, crc_in=None):
    import torch
    n = a.size
    nc = wm.num_chunks(n, chunk)
    ws = wm.new_workspace(n, chunk)
    wire = torch.full((wm.wire_bound(n, chunk),), 0xEE, dtype=torch.uint8, device="cuda")
    crc = torch.zeros(nc, dtype=torch.int32, device="cuda") if crc_in is None else torch.from_numpy(
        crc_in.view(np.int32).copy()).cuda()
    res = wm.new_result()
    d = None if dirty is None else torch.from_numpy(dirty).cuda()
    wm.wm_encode(torch.from_numpy(a).cuda(), chunk, d, crc, wire, ws, res)
    r = wm.read_result(res)
    return wire, crc.cpu().numpy().view(np.uint32), r, ws


def _run_decode(wm, wire_np, n, chunk, dst=None, dst_crc=None, strict=False):
    import torch
    nc = wm.num_chunks(n, chunk)
    ws = wm.new_workspace(n, chunk)
    wire = torch.from_numpy(np.ascontiguousarray(wire_np)).cuda()
    out = torch.full((n,), 0x5A, dtype=torch.uint8, device="cuda") if dst is None else torch.from_numpy(dst.copy()).cuda()
    crc = torch.zeros(nc, dtype=torch.int32, device="cuda") if dst_crc is None else torch.from_numpy(
        dst_crc.view(np.int32).copy()).cuda()
    res = wm.new_result()
    fn = wm.wm_decode_verify_strict if strict else wm.wm_decode_verify
    fn(wire, wire_np.size, out, chunk, crc, ws, res)
    return out.cpu().numpy(), crc.cpu().numpy().view(np.uint32), wm.read_result(res)


SIZES = [(TILE, TILE), (TILE + 3, TILE), (2 * TILE, 2 * TILE), (7 * TILE + 1234, 2 * TILE), (6 * TILE, 4 * TILE),
         (37 * TILE + 2, 4 * TILE), (64 * TILE, 16 * TILE)]


@pytest.mark.parametrize("n,chunk", SIZES)
def test_ent_images_match_the_oracle_bit_for_bit(wm, n, chunk):
    a = _mixed_cache(n, n % 1000)
    want, want_crc, want_res = oracle.encode(a, chunk, entropy=True)
    wire, crc, r, _ = _run_encode(wm, a, chunk)
    assert r.status == 0 and r.wire_len == want_res.wire_len and r.cache_crc == want_res.cache_crc
    got = wire[: r.wire_len].cpu().numpy()
    assert np.array_equal(got, want)
    assert np.array_equal(crc, want_crc)
    out, dcrc, rd = _run_decode(wm, got, n, chunk)
    assert rd.status == 0 and np.array_equal(out, a) and np.array_equal(dcrc, want_crc)
    out, dcrc, rd = _run_decode(wm, got, n, chunk, strict=True)
    assert rd.status == 0 and np.array_equal(out, a) and np.array_equal(dcrc, want_crc)


def test_ent_with_a_dirty_mask(wm):
    n, chunk = 24 * TILE + 100, 2 * TILE
    a = _mixed_cache(n, 3)
    nc = oracle.num_chunks(n, chunk)
    dirty = (np.arange(nc) % 3 != 1).astype(np.uint8)
    crc_in = oracle.checksum(a, chunk)
    want, want_crc, want_res = oracle.encode(a, chunk, dirty=dirty, crc_in=crc_in, entropy=True)
    wire, crc, r, _ = _run_encode(wm, a, chunk, dirty=dirty, crc_in=crc_in)
    got = wire[: r.wire_len].cpu().numpy()
    assert r.status == 0 and np.array_equal(got, want) and struct.unpack_from("<H", got, 6)[0] == 5
    base = a.copy()
    out, dcrc, rd = _run_decode(wm, got, n, chunk, dst=base, dst_crc=crc_in)
    assert rd.status == 0 and np.array_equal(out, a)


def test_ent_configs_round_trip_and_ratio(wm):
    from paper_2607_10389_b200 import inputs
    for name in ("tiny", "engine_small"):
        cfg = inputs.CONFIGS[name]
        a = inputs.make_cache(cfg).numpy().view(np.uint8).reshape(-1)
        want, want_crc, want_res = oracle.encode(a, cfg.chunk_bytes, entropy=True)
        wire, crc, r, _ = _run_encode(wm, a, cfg.chunk_bytes)
        got = wire[: r.wire_len].cpu().numpy()
        assert r.status == 0 and np.array_equal(got, want)
        assert r.wire_len < 0.71 * a.size                   # bit-plane packing gives 0.75 on these
        out, dcrc, rd = _run_decode(wm, got, a.size, cfg.chunk_bytes)
        assert rd.status == 0 and np.array_equal(out, a)


def test_ent_damage_verdicts_match_the_oracle(wm):
    n, chunk = 8 * TILE, 2 * TILE
    a = _gauss(n // 2, 9).view(np.uint8)
    wire, _, _ = oracle.encode(a, chunk, entropy=True)
    me = oracle.meta_end(n, chunk)
    entries = wire[64 + 16 * 4: 64 + 16 * 4 + 16].view("<u2")
    offs = np.concatenate([[0], np.cumsum(32 * (entries & 0x7FFF).astype(np.int64))])
    cases = []
    w = wire.copy(); w[me + 8] ^= 16; cases.append(w)                                # structure (count vs entry)
    w = wire.copy(); c = w[me + 8: me + 24].view("<u2"); c[0] += 1; c[1] -= 1; cases.append(w)      # streams do not fit
    w = wire.copy(); o = me + int(offs[5]); c = w[o + 8: o + 24].view("<u2"); c[6] += 2; c[7] -= 2; cases.append(w)
    w = wire.copy(); c = w[me + 8: me + 24].view("<u2"); c[3] = 40; cases.append(w)   # count out of range
    for k in (0, 1, 5, 77, 300, 1001, 2999):                                           # bits inside streams
        w = wire.copy(); w[me + int(offs[3]) + 8256 + k] ^= 1 << (k % 8); cases.append(w)
    w = wire.copy(); w[me + 100] ^= 4; cases.append(w)                                 # sign-mantissa byte
    w = wire.copy(); w[me + 3] ^= 1; cases.append(w)                                   # an anchor
    w = wire[:-32].copy(); cases.append(w)                                             # truncated
    live = np.full(n, 0x42, dtype=np.uint8)
    live_crc = np.arange(4, dtype=np.uint32)
    seen = set()
    for w in cases:
        want_out, want_crc, want = oracle.decode_verify(w, n, chunk, dst=live, dst_crc=live_crc, expect_entropy=True)
        out, dcrc, r = _run_decode(wm, w, n, chunk, dst=live, dst_crc=live_crc)
        assert (r.status, r.first_bad_chunk, r.n_bad_chunks) == (want.status, want.first_bad_chunk, want.n_bad_chunks)
        assert np.array_equal(dcrc, live_crc) and want.status != 0
        out, dcrc, r = _run_decode(wm, w, n, chunk, dst=live, dst_crc=live_crc, strict=True)
        assert r.status == want.status and np.array_equal(out, live) and np.array_equal(dcrc, live_crc)
        seen.add(want.status_name)
    assert {"ERR_STRUCT", "ERR_DESC", "ERR_CHUNK_CRC", "ERR_FORMAT"} <= seen


def test_option_and_image_must_agree(wm):
    n, chunk = 4 * TILE, 2 * TILE
    a = _gauss(n // 2, 10).view(np.uint8)
    w_ent, _, _ = oracle.encode(a, chunk, entropy=True)
    w_pack, _, _ = oracle.encode(a, chunk)
    _, _, r = _run_decode(wm, w_pack, n, chunk)                    # option on, default image
    assert r.status_name == "ERR_FORMAT" == oracle.decode_verify(w_pack, n, chunk, expect_entropy=True)[2].status_name
    wm.entropy_enable(False)
    _, _, r = _run_decode(wm, w_ent, n, chunk)                     # option off, ENT image
    assert r.status_name == "ERR_FORMAT" == oracle.decode_verify(w_ent, n, chunk, expect_entropy=False)[2].status_name
    out, _, r = _run_decode(wm, w_pack, n, chunk)
    assert r.status == 0 and np.array_equal(out, a)
    # and the default encoder is what it was
    import torch
    wire, crc, r, _ = _run_encode(wm, a, chunk)
    assert np.array_equal(wire[: r.wire_len].cpu().numpy(), w_pack)


def test_ent_leaves(wm):
    import torch
    n, chunk = 12 * TILE, 2 * TILE
    a = _mixed_cache(n, 17)
    want, want_crc, _ = oracle.encode(a, chunk, entropy=True)
    sizes = [4 * TILE, 2 * TILE, 6 * TILE]
    leaves, o = [], 0
    for sz in sizes:
        leaves.append(torch.from_numpy(a[o:o + sz].copy()).cuda()); o += sz
    nc = wm.num_chunks(n, chunk)
    ws = wm.new_workspace(n, chunk)
    wire = torch.empty(wm.wire_bound(n, chunk), dtype=torch.uint8, device="cuda")
    crc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    res = wm.new_result()
    wm.wm_encode_leaves(wm.make_leaf_table(leaves), n, chunk, None, crc, wire, ws, res)
    r = wm.read_result(res)
    assert r.status == 0 and np.array_equal(wire[: r.wire_len].cpu().numpy(), want)
    dst = [torch.zeros_like(x) for x in leaves]
    dcrc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    wm.wm_decode_verify_leaves(wire, r.wire_len, wm.make_leaf_table(dst), n, chunk, dcrc, ws, res)
    assert wm.read_result(res).status == 0 and all(torch.equal(x, y) for x, y in zip(leaves, dst))


def test_both_options_in_one_image(wm):
    """Zero and constant tiles as table entries, the rest in the shortest of ENT, PACK and raw."""
    n, chunk = 10 * TILE, 2 * TILE
    a = _mixed_cache(n, 23)
    a[6 * TILE:8 * TILE] = 0
    a[8 * TILE:9 * TILE].view("<u2")[:] = 0xFF80
    w, crc, res = oracle.encode(a, chunk, zero_tiles=True, entropy=True)
    assert struct.unpack_from("<H", w, 6)[0] == 6
    entries = w[64 + 16 * 5: 64 + 16 * 5 + 20].view("<u2")
    assert list(entries[6:9]) == [1, 1, 2] and entries[0] & 0x8000 and entries[1] == 512
    out, dcrc, r = _run_decode(wm, w, n, chunk)
    assert r.status == 0 and np.array_equal(out, a) and np.array_equal(dcrc, crc)
    wm.zero_tiles_enable(True)
    try:
        wire, crc2, r2, _ = _run_encode(wm, a, chunk)
    finally:
        wm.zero_tiles_enable(False)
    assert r2.status == 0 and np.array_equal(wire[: r2.wire_len].cpu().numpy(), w) and np.array_equal(crc2, crc)


def test_regular_tiles_keep_their_bit_planes(wm):
    """The option never lengthens an image: tiles whose bit planes are shorter than their ENT form
    (one exponent, two exponents, narrow ranges) stay PACK tiles inside an image with the option."""
    rng = np.random.default_rng(8)
    tiles = [np.full(8192, 0x3F80, dtype="<u2"),
             ((np.arange(8192) % 2 + 126) << 7).astype("<u2"),
             _gauss(8192, 51),
             ((rng.integers(100, 104, 8192) << 7) | rng.integers(0, 128, 8192)).astype("<u2"),
             rng.integers(0, 65536, 8192).astype("<u2"),
             _gauss(8192, 52, 1e-3)]
    a = np.concatenate(tiles).view(np.uint8)
    n, chunk = a.size, 2 * TILE
    want, want_crc, want_res = oracle.encode(a, chunk, entropy=True)
    plain, _, plain_res = oracle.encode(a, chunk)
    entries = want[64 + 16 * 3: 64 + 16 * 3 + 12].view("<u2")
    assert [int(e) & 0x8000 != 0 for e in entries] == [False, False, True, False, False, True]
    assert want_res.wire_len < plain_res.wire_len
    wire, crc, r, _ = _run_encode(wm, a, chunk)
    got = wire[: r.wire_len].cpu().numpy()
    assert r.status == 0 and np.array_equal(got, want) and np.array_equal(crc, want_crc)
    for strict in (False, True):
        out, dcrc, rd = _run_decode(wm, got, n, chunk, strict=strict)
        assert rd.status == 0 and np.array_equal(out, a) and np.array_equal(dcrc, want_crc)
    # a damaged descriptor of a PACK tile inside such an image is found like in any other image
    me = oracle.meta_end(n, chunk)
    bad = want.copy()
    bad[me + 1] ^= 0x10
    want_bad = oracle.decode_verify(bad, n, chunk, expect_entropy=True)[2]
    _, _, rb = _run_decode(wm, bad, n, chunk)
    assert (rb.status, rb.first_bad_chunk, rb.n_bad_chunks) == (want_bad.status, want_bad.first_bad_chunk, want_bad.n_bad_chunks)
    assert want_bad.status_name == "ERR_DESC"


def test_ent_repeatable_under_load(wm):
    """Placement is decided by whichever team gets there first; the bytes must not depend on it."""
    import torch
    from paper_2607_10389_b200 import inputs
    cfg = inputs.CONFIGS["engine_small"]
    a = inputs.make_cache(cfg).numpy().view(np.uint8).reshape(-1)
    first = None
    for _ in range(25):
        wire, crc, r, _ = _run_encode(wm, a, cfg.chunk_bytes)
        got = wire[: r.wire_len].clone()
        if first is None:
            first = got
        assert r.status == 0 and torch.equal(got, first)
        out, _, rd = _run_decode(wm, got.cpu().numpy(), a.size, cfg.chunk_bytes)
        assert rd.status == 0 and np.array_equal(out, a)


def test_bits_that_carry_no_data_are_checked_like_the_oracle_checks_them(wm):
    """An image with an ENT tile, a CONST tile, a ZERO tile and a ragged tail.  Every bit of the
    metadata, of the ENT tile's header, of its last 64 bytes (the end fill), of the CONST tile's 32
    bytes, and a sample of all the others is flipped in turn; each time the verdict (status, first
    bad chunk, count) is the oracle's, and it is never OK."""
    import torch
    a = np.concatenate([_gauss(TILE // 2, 31).view(np.uint8), np.full(8192, 0xFF80, "<u2").view(np.uint8),
                        np.zeros(TILE, np.uint8), _gauss(150, 32).view(np.uint8)])
    n, chunk = a.size, 4 * TILE
    want_wire, _, want = oracle.encode(a, chunk, zero_tiles=True, entropy=True)
    opt = wm.OPT_ZERO_TILES | wm.OPT_ENTROPY
    ws, res = wm.new_workspace(n, chunk), wm.new_result()
    wire = torch.zeros(wm.wire_bound(n, chunk), dtype=torch.uint8, device="cuda")
    crc = torch.zeros(1, dtype=torch.int32, device="cuda")
    wm.wm_encode_opt(torch.from_numpy(a).cuda(), chunk, None, crc, wire, ws, res, opt)
    r = wm.read_result(res)
    assert r.ok and np.array_equal(wire[: r.wire_len].cpu().numpy(), want_wire)
    me = oracle.meta_end(n, chunk)
    ent_len = 32 * (int(want_wire[64 + 16: 64 + 18].view(np.uint16)[0]) & 0x7FFF)
    bits = set(range(me * 8)) | set(range(me * 8, (me + 64) * 8)) | set(range((me + ent_len - 64) * 8, (me + ent_len + 32) * 8))
    rng = np.random.default_rng(3)
    bits |= set(int(b) for b in rng.integers(0, r.wire_len * 8, 1500))
    dst = torch.zeros(n, dtype=torch.uint8, device="cuda")
    dcrc = torch.zeros(1, dtype=torch.int32, device="cuda")
    for bit in sorted(bits):
        wire[bit // 8] ^= 1 << (bit % 8)
        wm.wm_decode_verify_opt(wire, r.wire_len, dst, chunk, dcrc, ws, res, wm.OPT_ENTROPY)
        rd = wm.read_result(res)
        w = want_wire.copy()
        w[bit // 8] ^= 1 << (bit % 8)
        o = oracle.decode_verify(w, n, chunk, expect_entropy=True)[2]
        assert rd.status != 0 and (rd.status, rd.first_bad_chunk, rd.n_bad_chunks) == (o.status, o.first_bad_chunk, o.n_bad_chunks), bit
        wire[bit // 8] ^= 1 << (bit % 8)
    wm.wm_decode_verify_opt(wire, r.wire_len, dst, chunk, dcrc, ws, res, wm.OPT_ENTROPY)
    assert wm.read_result(res).ok and np.array_equal(dst.cpu().numpy(), a)
