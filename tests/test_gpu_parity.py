"""Parity of the CUDA path (through the C ABI) with the CPU oracle: bit-exact checksums, dirty
masks, wire images and decoded caches on the same seeded inputs.  Tolerance 0 everywhere."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_10389_b200 import inputs

pytestmark = pytest.mark.gpu
TILE = 16384


@pytest.fixture(scope="module")
def G():
    from gpu_util import Gpu
    return Gpu


def _special_cache(n, seed):
    """Random bytes with a compressible first tile that holds NaN / Inf / denormal / -0 patterns."""
    rng = np.random.default_rng(seed)
    a = rng.integers(0, 256, n, dtype=np.uint8)
    if n >= TILE:
        v = rng.integers(0x3E00, 0x4100, 8192).astype("<u2")
        v[:6] = [0x7FC0, 0xFF80, 0x0001, 0x8000, 0x7F80, 0x0000]
        v[256:512] = 0x8000
        a[:TILE] = v.view(np.uint8)
    if n >= 3 * TILE:      # a tile with wide and narrow groups mixed
        v = (rng.integers(0, 128, 8192) | (rng.integers(100, 104, 8192) << 7)).astype("<u2")
        v[512:768] = (rng.integers(0, 128, 256) | (rng.integers(1, 250, 256) << 7)).astype("<u2")
        v[1024:1280] = 0x3F80
        a[2 * TILE:3 * TILE] = v.view(np.uint8)
    return a


SIZES = [1, 2, 3, 4, 5, 15, 16, 17, 4095, TILE - 1, TILE, TILE + 1, TILE + 3, 2 * TILE, 3 * TILE + 5536,
         2 * 65536 + 777, 5 * 65536]


@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("chunk", [TILE, 65536])
def test_checksum_ragged_sizes(G, n, chunk):
    from gpu_util import to_dev
    a = _special_cache(n, n)
    got = G(n, chunk).checksum(to_dev(a))
    assert np.array_equal(got, oracle.checksum(a, chunk))


@pytest.mark.parametrize("name", ["tiny", "tiny8m", "engine_small"])
def test_checksum_configs(G, name):
    cfg = inputs.CONFIGS[name]
    a = inputs.make_cache(cfg)
    got = G(cfg.nbytes, cfg.chunk_bytes).checksum(a.cuda())
    assert np.array_equal(got, oracle.checksum(a.numpy(), cfg.chunk_bytes))


@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("chunk", [TILE, 65536])
def test_encode_decode_ragged_sizes(G, n, chunk):
    from gpu_util import same_result, to_dev
    a = _special_cache(n, 1000 + n)
    g = G(n, chunk)
    want_wire, want_crc, want_res = oracle.encode(a, chunk)
    wire, crc, res, wire_dev = g.encode(to_dev(a))
    assert same_result(res, want_res), (res, want_res)
    assert np.array_equal(crc, want_crc)
    assert np.array_equal(wire[: res.wire_len], want_wire)
    out, dcrc, r = g.decode(wire_dev, res.wire_len)
    want_out, want_dcrc, want_r = oracle.decode_verify(want_wire, n, chunk)
    assert same_result(r, want_r), (r, want_r)
    assert r.status == 0 and np.array_equal(out, a) and np.array_equal(dcrc, want_dcrc)


@pytest.mark.parametrize("name", ["tiny", "tiny8m", "engine_small"])
def test_encode_decode_configs(G, name):
    from gpu_util import same_result
    cfg = inputs.CONFIGS[name]
    a = inputs.make_cache(cfg)
    g = G(cfg.nbytes, cfg.chunk_bytes)
    want_wire, want_crc, want_res = oracle.encode(a.numpy(), cfg.chunk_bytes)
    wire, crc, res, wire_dev = g.encode(a.cuda())
    assert same_result(res, want_res), (res, want_res)
    assert np.array_equal(crc, want_crc)
    assert np.array_equal(wire[: res.wire_len], want_wire)
    out, dcrc, r = g.decode(wire_dev, res.wire_len)
    assert r.status == 0 and np.array_equal(out, a.numpy()) and np.array_equal(dcrc, want_crc)
    # the oracle decodes the GPU's image and the GPU decodes the oracle's
    assert np.array_equal(oracle.decode_verify(wire[: res.wire_len], cfg.nbytes, cfg.chunk_bytes)[0], a.numpy())


def test_all_group_widths_and_orders(G):
    """Every width 0..8 in every group position, elements distinguishable by position."""
    from gpu_util import to_dev
    rng = np.random.default_rng(99)
    tiles = []
    for rot in range(9):
        E = np.zeros(8192, dtype=np.uint32)
        for g in range(32):
            w = (g + rot) % 9
            base = rng.integers(0, 256 - (1 << w) + 1) if w else rng.integers(0, 256)
            d = rng.integers(0, 1 << w, 256) if w else np.zeros(256, dtype=np.int64)
            if w:
                d[rng.integers(0, 256)] = 0
                d[rng.integers(1, 256)] = (1 << w) - 1
                d[0] = 0
            E[g * 256:(g + 1) * 256] = base + d
        SM = rng.integers(0, 256, 8192).astype(np.uint32)
        v = ((SM & 1) << 15) | (E << 7) | (SM >> 1)
        tiles.append(v.astype("<u2").view(np.uint8))
    a = np.concatenate(tiles)
    for chunk in (TILE, 4 * TILE):
        g = G(len(a), chunk)
        want_wire, want_crc, want_res = oracle.encode(a, chunk)
        wire, crc, res, wire_dev = g.encode(to_dev(a))
        assert res.wire_len == want_res.wire_len
        assert np.array_equal(wire[: res.wire_len], want_wire)
        out, _, r = g.decode(wire_dev, res.wire_len)
        assert r.status == 0 and np.array_equal(out, a)


def test_incompressible_takes_raw_path(G):
    from gpu_util import to_dev
    rng = np.random.default_rng(3)
    n, chunk = 40 * TILE, 8 * TILE
    a = rng.integers(0, 256, n, dtype=np.uint8)
    g = G(n, chunk)
    wire, crc, res, wire_dev = g.encode(to_dev(a))
    me = oracle.meta_end(n, chunk)
    assert res.wire_len == me + n
    assert np.array_equal(wire[:res.wire_len], oracle.encode(a, chunk)[0])
    out, _, r = g.decode(wire_dev, res.wire_len)
    assert r.status == 0 and np.array_equal(out, a)
    # one injected bit flip must be rejected
    flipped = wire_dev.clone()
    flipped[me + 12345] ^= 0x20
    _, _, r = g.decode(flipped, res.wire_len)
    assert r.status_name == "ERR_CHUNK_CRC" and r.n_bad_chunks == 1 and r.first_bad_chunk == 12345 // chunk


def test_dirty_diff_and_precopy_round(G):
    from gpu_util import same_result
    cfg = inputs.CONFIGS["tiny"]
    prev = inputs.make_cache(cfg)
    cur, rewritten = inputs.rewrite_random_chunks(prev, cfg.chunk_bytes, 0.75, seed=77)
    g = G(cfg.nbytes, cfg.chunk_bytes)
    dirty, idx, n = g.dirty_diff(cur.cuda(), prev.cuda())
    want_dirty, want_idx = oracle.dirty_diff(cur.numpy(), prev.numpy(), cfg.chunk_bytes)
    assert np.array_equal(dirty, want_dirty) and np.array_equal(idx, want_idx) and n == 24
    assert np.array_equal(dirty, rewritten.numpy())
    # without an index list
    d2, _, n2 = g.dirty_diff(cur.cuda(), prev.cuda(), want_idx=False)
    assert np.array_equal(d2, want_dirty) and n2 == 24
    # identical snapshots: nothing dirty, and a masked encode of nothing is an empty payload
    d0, i0, n0 = g.dirty_diff(prev.cuda(), prev.clone().cuda())
    assert n0 == 0 and not d0.any()
    crc_prev = g.checksum(prev.cuda())
    w0, _, r0, w0_dev = g.encode(prev.cuda(), dirty=d0, crc_in=crc_prev)
    want_w0, _, want_r0 = oracle.encode(prev.numpy(), cfg.chunk_bytes, dirty=d0, crc_in=crc_prev)
    assert same_result(r0, want_r0) and r0.payload_bytes == 0 and np.array_equal(w0[: r0.wire_len], want_w0)
    # the round: encode dirty chunks only, install over the previous snapshot
    wire, crc, res, wire_dev = g.encode(cur.cuda(), dirty=dirty, crc_in=crc_prev)
    want_wire, want_crc, want_res = oracle.encode(cur.numpy(), cfg.chunk_bytes, dirty=want_dirty, crc_in=crc_prev)
    assert same_result(res, want_res) and np.array_equal(crc, want_crc)
    assert np.array_equal(wire[: res.wire_len], want_wire)
    out, dcrc, r = g.decode(wire_dev, res.wire_len, dst=prev, dst_crc=crc_prev)
    assert r.status == 0 and np.array_equal(out, cur.numpy())
    assert np.array_equal(dcrc, oracle.checksum(cur.numpy(), cfg.chunk_bytes))
    # a destination whose clean chunk is not the source's is refused, its CRC vector untouched
    stale = crc_prev.copy()
    clean = int(np.nonzero(want_dirty == 0)[0][2])
    stale[clean] ^= 0x40
    _, dcrc, r = g.decode(wire_dev, res.wire_len, dst=prev, dst_crc=stale)
    want_r = oracle.decode_verify(want_wire, cfg.nbytes, cfg.chunk_bytes, dst=prev.numpy(), dst_crc=stale)[2]
    assert same_result(r, want_r) and r.status_name == "ERR_STALE" and np.array_equal(dcrc, stale)


def test_dirty_diff_single_bytes_and_ragged_tail(G):
    from gpu_util import to_dev
    rng = np.random.default_rng(31)
    chunk, n = 65536, 65536 * 5 + 16384 + 7
    a = rng.integers(0, 256, n, dtype=np.uint8)
    g = G(n, chunk)
    for pos in (0, chunk - 1, chunk, 3 * chunk + 40000, 5 * chunk + 16383, n - 1, n - 7, n - 8):
        b = a.copy()
        b[pos] ^= 0x01
        dirty, idx, cnt = g.dirty_diff(to_dev(b), to_dev(a))
        want = np.zeros(6, dtype=np.uint8)
        want[pos // chunk] = 1
        assert np.array_equal(dirty, want) and idx.tolist() == [pos // chunk] and cnt == 1, pos
    b = a.copy()
    for c in (0, 2, 5):
        b[c * chunk + 5] ^= 0xFF
    dirty, idx, cnt = g.dirty_diff(to_dev(b), to_dev(a))
    assert idx.tolist() == [0, 2, 5] and cnt == 3


def _flip_cases(wire_len, me, rng, n_payload):
    bits = [8 * 0 + 1, 8 * 5, 8 * 6 + 3, 8 * 9, 8 * 17, 8 * 21, 8 * 25, 8 * 28 + 2, 8 * 33, 8 * 41, 8 * 48, 8 * 53, 8 * 60]
    bits += rng.integers(64 * 8, me * 8, 40).tolist()                    # directory, tile table, pad
    bits += rng.integers(me * 8, (me + 64) * 8, 40).tolist()             # descriptors of the first tile
    bits += rng.integers((me + 64) * 8, wire_len * 8, n_payload).tolist()
    bits.append(wire_len * 8 - 1)
    return bits


def test_single_bit_flips_match_oracle_verdicts(G):
    from gpu_util import same_result, to_dev
    rng = np.random.default_rng(21)
    n = 6 * TILE + 300
    v = rng.integers(0x3C00, 0x4080, n // 2).astype("<u2")
    a = v.view(np.uint8).copy()
    a[2 * TILE:3 * TILE] = rng.integers(0, 256, TILE, dtype=np.uint8)     # one RAW tile
    chunk = 2 * TILE
    g = G(n, chunk)
    wire, crc, res, wire_dev = g.encode(to_dev(a))
    want_wire = oracle.encode(a, chunk)[0]
    assert np.array_equal(wire[: res.wire_len], want_wire)
    me = oracle.meta_end(n, chunk)
    live = to_dev(np.full(n, 0x11, dtype=np.uint8))
    for bit in _flip_cases(res.wire_len, me, rng, 120):
        w = wire_dev.clone()
        w[bit // 8] ^= (1 << (bit % 8))
        _, dcrc, r = g.decode(w, res.wire_len)
        hw = want_wire.copy()
        hw[bit // 8] ^= 1 << (bit % 8)
        want_r = oracle.decode_verify(hw, n, chunk)[2]
        assert r.status != 0, bit
        assert same_result(r, want_r), (bit, r, want_r)
        assert not dcrc.any()
    assert (live.cpu().numpy() == 0x11).all()      # the live buffer is never the decoder's target


def test_unsound_descriptors_keep_the_decoder_inside_its_stage(G):
    """Descriptor blocks overwritten wholesale (all ones: width 15 in every group; widths 8 and
    valid check bits throughout: a sum the tile cannot have; random bytes): the verdict is the
    oracle's, nothing faults, the destination's checksums stay as they were and the next call on
    the same workspace decodes the untouched image.  (Only one warp of a team judges the
    descriptors; the others read whatever widths they find, clamped so that they stay in bounds.)"""
    from gpu_util import same_result, to_dev
    rng = np.random.default_rng(33)
    n = 9 * TILE + 1000
    v = (rng.normal(size=n // 2) * 3.0).astype(np.float32)
    a = (v.view(np.uint32) >> 16).astype("<u2").view(np.uint8).copy()
    chunk = 4 * TILE
    g = G(n, chunk)
    wire, crc, res, wire_dev = g.encode(to_dev(a))
    want_wire = oracle.encode(a, chunk)[0]
    assert np.array_equal(wire[: res.wire_len], want_wire)
    me = oracle.meta_end(n, chunk)
    tab = np.frombuffer(want_wire[64 + 16 * oracle.num_chunks(n, chunk): me].tobytes(), dtype="<u2")[: oracle.num_tiles(n)]
    starts = me + np.concatenate([[0], np.cumsum([32 * int(e) if e < 0xFFFF else n % TILE for e in tab])[:-1]])
    packed = [i for i, e in enumerate(tab) if 258 <= e < 512]
    assert len(packed) >= 8

    def desc_word(base, w):
        return base | (w << 8) | ((((base & 15) ^ (base >> 4) ^ w ^ 5) & 15) << 12)

    blocks = {
        "all ones": np.full(64, 0xFF, np.uint8),
        "width 8 everywhere, check bits right": np.array([desc_word(100, 8)] * 32, dtype="<u2").view(np.uint8),
        "width 15 with matching check bits": np.array([desc_word(7, 15)] * 32, dtype="<u2").view(np.uint8),
        "random": rng.integers(0, 256, 64, dtype=np.uint8),
    }
    for name, block in blocks.items():
        for t in (packed[0], packed[len(packed) // 2], packed[-1]):
            hw = want_wire.copy()
            hw[starts[t]: starts[t] + 64] = block
            want_r = oracle.decode_verify(hw, n, chunk)[2]
            assert want_r.status_name in ("ERR_DESC", "ERR_STRUCT"), (name, t, want_r.status_name)
            _, dcrc, r = g.decode(to_dev(np.concatenate([hw, np.zeros((-hw.size) % 16, np.uint8)])), res.wire_len)
            assert same_result(r, want_r), (name, t, r, want_r)
            assert not dcrc.any()
    out, dcrc, r = g.decode(wire_dev, res.wire_len)
    assert r.ok and np.array_equal(out, a) and np.array_equal(dcrc, crc)


def test_truncation_extension_wrong_arguments(G):
    from gpu_util import same_result, to_dev
    rng = np.random.default_rng(5)
    n, chunk = 4 * TILE + 100, 2 * TILE
    a = rng.integers(0x3C, 0x41, n, dtype=np.uint8)
    g = G(n, chunk)
    wire, _, res, wire_dev = g.encode(to_dev(a))
    for wl in (res.wire_len - 1, res.wire_len + 1, 40, 64, 0):
        _, _, r = g.decode(wire_dev, wl)
        assert r.status_name == "ERR_FORMAT", wl
    # the same image decoded under another geometry
    g2 = G(n + 2, chunk)
    assert g2.decode(wire_dev, res.wire_len)[2].status_name == "ERR_FORMAT"
    g3 = G(n, 4 * TILE)
    assert g3.decode(wire_dev, res.wire_len)[2].status_name == "ERR_FORMAT"


def test_capacity_error_and_argument_errors(G):
    from gpu_util import to_dev
    from paper_2607_10389_b200 import binding as wm
    rng = np.random.default_rng(6)
    n, chunk = 8 * TILE, 2 * TILE
    a = rng.integers(0, 256, n, dtype=np.uint8)
    g = G(n, chunk)
    full = g.encode(to_dev(a))[2]
    _, _, r, _ = g.encode(to_dev(a), wire_cap=full.wire_len - 32)
    assert r.status_name == "ERR_CAPACITY" and r.wire_len == full.wire_len
    _, _, r, _ = g.encode(to_dev(a), wire_cap=full.wire_len)
    assert r.status == 0
    with pytest.raises(wm.WmError):
        g.encode(to_dev(a), wire_cap=oracle.meta_end(n, chunk) - 1)
    with pytest.raises(wm.WmError):
        G(n, chunk).checksum(to_dev(a)[1:])            # not 16-byte aligned
    assert wm.workspace_bytes(n, 1000) == 0
    with pytest.raises(wm.WmError):
        wm.wm_checksum(to_dev(a), 1000, torch.zeros(4, dtype=torch.int32, device="cuda"), g.ws)


def test_repeatable_bytes(G):
    """The wire image is canonical: repeated runs give identical bytes."""
    cfg = inputs.CONFIGS["tiny8m"]
    a = inputs.make_cache(cfg).cuda()
    g = G(cfg.nbytes, cfg.chunk_bytes)
    w1, _, r1, _ = g.encode(a)
    w2, _, r2, _ = g.encode(a)
    assert r1.wire_len == r2.wire_len and np.array_equal(w1[: r1.wire_len], w2[: r2.wire_len])


@pytest.mark.gpu
@pytest.mark.parametrize("layout", ["some", "all", "first_of_chunk", "masked"])
def test_zero_tiles_match_the_oracle(layout):
    """Tiles of all-zero bytes (unused allocation) become table entries without payload."""
    from gpu_util import Gpu, same_result, to_dev
    rng = np.random.default_rng(11)
    chunk = 4 * TILE
    nt = 13
    n = nt * TILE + 700
    a = (rng.normal(size=(n + 1) // 2).astype(np.float32).view(np.uint32) >> 16).astype("<u2").view(np.uint8)[:n].copy()
    zero = {"some": [1, 2, 6, 11], "all": list(range(nt)), "first_of_chunk": [0, 4, 8, 12], "masked": [1, 5, 6, 7]}[layout]
    for t in zero:
        a[t * TILE:(t + 1) * TILE] = 0
    if layout == "all":
        a[nt * TILE:] = 0
    a[3 * TILE + 10:3 * TILE + 12] = (0, 0x80) if layout != "all" else (0, 0)      # a minus zero stays data
    nc = (n + chunk - 1) // chunk
    dirty = (np.arange(nc) % 2 == 1).astype(np.uint8) if layout == "masked" else None
    crc_in = np.full(nc, 0x12345678, dtype=np.uint32)
    from paper_2607_10389_b200 import binding as wm
    want_wire, want_crc, want = oracle.encode(a, chunk, dirty=dirty, crc_in=crc_in, zero_tiles=True)
    plain_wire, _, plain = oracle.encode(a, chunk, dirty=dirty, crc_in=crc_in)
    g = Gpu(n, chunk)
    # without the option the zeros pack like any constant tile ...
    wire0, _, r0, _ = g.encode(to_dev(a), dirty=dirty, crc_in=crc_in)
    assert same_result(r0, plain) and np.array_equal(wire0[: r0.wire_len], plain_wire)
    # ... with it they are table entries
    wm.zero_tiles_enable(True)
    try:
        wire, crc, r, wire_dev = g.encode(to_dev(a), dirty=dirty, crc_in=crc_in)
    finally:
        wm.zero_tiles_enable(False)
    assert same_result(r, want) and r.wire_len < r0.wire_len
    assert np.array_equal(wire[: r.wire_len], want_wire) and np.array_equal(crc, want_crc)
    old = np.full(n, 0x5A, dtype=np.uint8)
    if dirty is not None:
        for c in np.nonzero(dirty == 0)[0]:
            old[c * chunk:(c + 1) * chunk] = a[c * chunk:(c + 1) * chunk]
    want_out, want_dcrc, want_r = oracle.decode_verify(want_wire, n, chunk, dst=old, dst_crc=want_crc)
    out, dcrc, rd = g.decode(wire_dev, r.wire_len, dst=old, dst_crc=want_crc)
    assert same_result(rd, want_r) and rd.ok
    assert np.array_equal(out, want_out) and np.array_equal(out, a) and np.array_equal(dcrc, want_dcrc)


@pytest.mark.parametrize("layout", ["mixed", "near_misses", "masked"])
def test_constant_tiles_match_the_oracle(layout):
    """The zero-tile option also ships a tile of one non-zero value (a mask fill) as entry 2 and
    32 bytes; tiles that are constant only per warp, per half-word or but for one element are data."""
    from gpu_util import Gpu, same_result, to_dev
    from paper_2607_10389_b200 import binding as wm
    rng = np.random.default_rng(12)
    chunk = 4 * TILE
    nt = 14
    n = nt * TILE + 300
    a = (rng.normal(size=(n + 1) // 2).astype(np.float32).view(np.uint32) >> 16).astype("<u2").view(np.uint8)[:n].copy()
    v = a.view("<u2") if n % 2 == 0 else a[:n - 1].view("<u2")

    def fill(t, value):
        v[t * 8192:(t + 1) * 8192] = value

    fill(1, 0xFF80)                       # -Inf
    fill(2, 0x3F80)                       # 1.0
    fill(5, 0x0001)                       # a denormal: exponent 0, not the zero tile
    fill(6, 0x8000)                       # minus zero: constant, not zero
    fill(9, 0)                            # zeros: entry 1 as before
    fill(12, 0x7FC0)                      # NaN
    if layout == "near_misses":
        fill(3, 0x3F80); v[3 * 8192 + 8191] = 0x3F81                   # one element off at the very end
        fill(4, 0x3F80); v[4 * 8192:4 * 8192 + 1024] = 0x3F00         # constant per warp, two values
        fill(7, 0x4000); v[7 * 8192 + 1::2] = 0x4001                  # the two halves of every word differ
        fill(8, 0x3F80); v[8 * 8192 + 4096] = 0xBF80                  # one sign flipped
        fill(10, 0x0000); v[10 * 8192 + 77] = 0x0080                  # zeros but one
    nc = (n + chunk - 1) // chunk
    dirty = (np.arange(nc) % 2 == 0).astype(np.uint8) if layout == "masked" else None
    crc_in = np.full(nc, 0xCAFE, dtype=np.uint32)
    want_wire, want_crc, want = oracle.encode(a, chunk, dirty=dirty, crc_in=crc_in, zero_tiles=True)
    tab = want_wire[64 + 16 * nc: 64 + 16 * nc + 2 * (nt + 1)].view("<u2")
    if layout == "mixed":
        assert [int(tab[t]) for t in (1, 2, 5, 6, 9, 12)] == [2, 2, 2, 2, 1, 2]
    if layout == "near_misses":
        assert all(int(tab[t]) >= 258 for t in (3, 4, 7, 8, 10))
    g = Gpu(n, chunk)
    wm.zero_tiles_enable(True)
    try:
        wire, crc, r, wire_dev = g.encode(to_dev(a), dirty=dirty, crc_in=crc_in)
    finally:
        wm.zero_tiles_enable(False)
    assert same_result(r, want)
    assert np.array_equal(wire[: r.wire_len], want_wire) and np.array_equal(crc, want_crc)
    old = np.full(n, 0x5A, dtype=np.uint8)
    if dirty is not None:
        for c in np.nonzero(dirty == 0)[0]:
            old[c * chunk:(c + 1) * chunk] = a[c * chunk:(c + 1) * chunk]
    want_out, want_dcrc, want_r = oracle.decode_verify(want_wire, n, chunk, dst=old, dst_crc=want_crc)
    out, dcrc, rd = g.decode(wire_dev, r.wire_len, dst=old, dst_crc=want_crc)
    assert same_result(rd, want_r) and rd.ok and np.array_equal(out, a) and np.array_equal(dcrc, want_dcrc)
    # a damaged value is caught by the chunk checksum; entry 2 without the option's flag is refused
    bad = want_wire.copy()
    me = oracle.meta_end(n, chunk)
    first_const = 32 * int(tab[0])                     # tile 0 is an ordinary packed tile; tile 1's value follows it
    if dirty is None:
        bad[me + first_const] ^= 0x40                  # tile 1's value (tile 0 comes first in the payload)
        want_bad = oracle.decode_verify(bad, n, chunk, dst=old, dst_crc=want_crc)[2]
        _, _, rb = g.decode(to_dev(bad), bad.size, dst=old, dst_crc=want_crc)
        assert same_result(rb, want_bad) and want_bad.status_name == "ERR_CHUNK_CRC"
