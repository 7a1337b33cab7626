"""Pins of the oracle's WM1 encoder / decoder: hand-built tiles, a size law recomputed
independently with numpy, the blueprint's worked example, round trips, and rejection of
every kind of damage."""
import os
import struct

import numpy as np
import pytest
import torch

import oracle
from paper_2607_10389_b200 import inputs

HERE = os.path.dirname(os.path.abspath(__file__))
TILE = 16384


def _hdr(wire):
    f = struct.unpack_from("<4sHHQIIIIQQII8s", wire.tobytes()[:64])
    keys = ("magic version flags nbytes chunk_bytes tile_bytes n_chunks n_present payload_bytes "
            "wire_len cache_crc meta_crc pad").split()
    return dict(zip(keys, f))


def _dir(wire, nc):
    raw = wire[64:64 + 16 * nc].tobytes()
    return [struct.unpack_from("<QII", raw, 16 * c) for c in range(nc)]


def _tab(wire, nc, nt):
    return np.frombuffer(wire[64 + 16 * nc:64 + 16 * nc + 2 * nt].tobytes(), dtype="<u2")


def _bf16_tile(E, SM=None):
    """Tile from exponents E[8192] and sign-mantissa bytes SM[8192] (memory order)."""
    E = np.asarray(E, dtype=np.uint32)
    SM = np.zeros(8192, dtype=np.uint32) if SM is None else np.asarray(SM, dtype=np.uint32)
    v = ((SM & 1) << 15) | (E << 7) | (SM >> 1)
    return v.astype("<u2").view(np.uint8)


def _coded(e):
    r, l, h = e // 64, (e % 64) // 2, e % 2
    return 8 * l + 2 * r + h


def test_geometry():
    assert oracle.meta_end(TILE, TILE) == 96          # 64 + 16 + 2 = 82 -> 96
    assert oracle.meta_end(1_671_168_000, 1 << 20) == 229_568
    assert oracle.meta_end(1 << 30, 1 << 20) == 147_520
    assert oracle.wire_bound(1 << 30, 1 << 20) == (1 << 30) + 147_520


def test_constant_tile_is_hand_checkable():
    # every element 0x3F80 (1.0): E = 127, SM = 0; all widths 0 -> 8256 bytes
    tile = np.tile(np.array([0x80, 0x3F], dtype=np.uint8), 8192)
    wire, crc, res = oracle.encode(tile, TILE)
    assert res.status == 0 and res.wire_len == 96 + 8256 and res.payload_bytes == 8256
    assert _tab(wire, 1, 1).tolist() == [258]
    body = wire[96:]
    chk = (127 & 0xF) ^ (127 >> 4) ^ 0 ^ 5
    assert body[:64].tolist() == [127, chk << 4] * 32
    assert not body[64:].any()
    h = _hdr(wire)
    assert (h["magic"], h["version"], h["flags"], h["nbytes"], h["chunk_bytes"], h["tile_bytes"]) == \
        (b"WMV1", 1, 0, TILE, TILE, TILE)
    assert (h["n_chunks"], h["n_present"], h["wire_len"], h["pad"]) == (1, 1, 96 + 8256, bytes(8))
    assert h["cache_crc"] == crc[0] == oracle.crc_bitwise(tile)
    assert _dir(wire, 1) == [(0, 8256, int(crc[0]))]
    meta = wire[:96].copy()
    meta[52:56] = 0
    assert h["meta_crc"] == oracle.crc_bitwise(meta)


def test_single_bit_of_exponent_plane_lands_where_the_format_says():
    # group 3: one element (memory index 5) has E = base + 1 -> w = 1, one bit set at coded position
    E = np.full(8192, 100)
    E[3 * 256 + 5] = 101
    SM = np.arange(8192) % 251
    tile = _bf16_tile(E, SM)
    wire, _, res = oracle.encode(tile, TILE)
    assert res.payload_bytes == 8256 + 32
    body = wire[96:]
    descs = np.frombuffer(body[:64].tobytes(), dtype="<u2")
    for g in range(32):
        w = 1 if g == 3 else 0
        assert descs[g] == 100 | (w << 8) | ((((100 & 0xF) ^ (100 >> 4) ^ w ^ 5) & 0xF) << 12)
    k = _coded(5)
    assert k == 17
    ep = body[64 + 8192:]
    want = np.zeros(32, dtype=np.uint8)
    want[k // 8] = 1 << (k % 8)
    assert ep.tolist() == want.tolist()
    # SM plane: byte 256 g + coded(e) holds SM of element e
    sm = body[64:64 + 8192]
    for g in (0, 3, 31):
        for e in (0, 1, 2, 63, 64, 65, 127, 128, 200, 255):
            assert sm[256 * g + _coded(e)] == SM[256 * g + e]


def test_wide_group_bit_layout():
    # group 0 spans exponents 7..7+200 -> w = 8; element e has d = e % 201
    E = np.full(8192, 7)
    E[:256] = 7 + (np.arange(256) * 37) % 201
    E[0] = 7
    E[1] = 207
    tile = _bf16_tile(E)
    wire, _, res = oracle.encode(tile, TILE)
    assert res.payload_bytes == 8256 + 32 * 8
    ep = wire[96 + 64 + 8192:]
    for e in range(256):
        assert ep[_coded(e)] == E[e] - 7


def _planes_python(d, w):
    """Bit planes of a group, built with Python integers: widths 4, 2, 1 present when the bit
    of w is set, consecutive bits of d from bit 0; element with coded position k at bits
    [k p, (k+1) p) of its p-bit plane."""
    if w == 8:
        widths = [8]
    else:
        widths = [p for p in (4, 2, 1) if w & p]
    out, lo = b"", 0
    for p in widths:
        bits = 0
        for e in range(256):
            bits |= ((int(d[e]) >> lo) & ((1 << p) - 1)) << (p * _coded(e))
        out += bits.to_bytes(32 * p, "little")
        lo += p
    return out


@pytest.mark.parametrize("w", [1, 2, 3, 4, 5, 6, 7, 8])
def test_group_bit_planes_against_python_integers(w):
    rng = np.random.default_rng(w)
    base = 0 if w == 8 else 50
    E = np.full(8192, base)
    d = rng.integers(0, 1 << w, 256)
    d[10], d[11] = 0, (1 << w) - 1
    E[5 * 256:6 * 256] = base + d
    wire, _, _ = oracle.encode(_bf16_tile(E), TILE)
    ep = wire[96 + 64 + 8192:]
    assert len(ep) == 32 * w
    assert ep.tobytes() == _planes_python(d, w)


def test_five_bit_group_planes_by_hand():
    # d = 0b10011 at memory element 7 only: nibble 3 in the 4-bit plane, bit 1 in the 1-bit plane
    E = np.full(8192, 60)
    E[7] = 60 + 0b10011
    wire, _, _ = oracle.encode(_bf16_tile(E), TILE)
    ep = wire[96 + 64 + 8192:]
    assert len(ep) == 160
    k = _coded(7)                       # r = 0, l = 3, h = 1 -> 25
    assert k == 25
    want = np.zeros(160, dtype=np.uint8)
    want[k // 2] = 0x3 << (4 * (k % 2))      # 4-bit plane, 128 bytes
    want[128 + k // 8] = 1 << (k % 8)        # 1-bit plane, 32 bytes
    assert ep.tolist() == want.tolist()


@pytest.mark.parametrize("d,length,want_bytes", [
    # One element differs from its group's base, memory element 201 of group 0: row 3, word 4, high
    # half, so coded position k = 8*4 + 2*3 + 1 = 39.  Bytes worked out on paper from the format text:
    # width 2 (d = 10b): one 2-bit plane; k = 39 sits at bits 78-79 = byte 9, bits 6-7
    (0b10, 64, {9: 0x80}),
    # width 3 (d = 101b): 2-bit plane takes bits 0-1 (01b), then the 1-bit plane (from byte 64) takes
    # bit 2: bit 39 = byte 4, bit 7
    (0b101, 96, {9: 0x40, 64 + 4: 0x80}),
    # width 6 (d = 101101b): 4-bit plane takes 1101b into the high nibble of byte 19 (k odd), the
    # 2-bit plane (from byte 128) takes 10b
    (0b101101, 192, {19: 0xD0, 128 + 9: 0x80}),
    # width 7 (d = 1011010b): 4-bit plane 1010b, 2-bit plane 01b, 1-bit plane (from byte 192) 1
    (0b1011010, 224, {19: 0xA0, 128 + 9: 0x40, 192 + 4: 0x80}),
])
def test_two_and_three_plane_groups_by_hand(d, length, want_bytes):
    E = np.full(8192, 60)
    E[201] = 60 + d
    wire, _, _ = oracle.encode(_bf16_tile(E), TILE)
    ep = wire[96 + 64 + 8192:]
    assert len(ep) == length
    want = np.zeros(length, dtype=np.uint8)
    for at, v in want_bytes.items():
        want[at] = v
    assert ep.tolist() == want.tolist()
    desc = struct.unpack_from("<H", wire, 96)[0]
    assert desc & 0xFF == 60 and (desc >> 8) & 15 == d.bit_length()


def test_raw_fallback_never_expands_beyond_metadata():
    rng = np.random.default_rng(2)
    n, chunk = 8 * TILE, 4 * TILE
    a = rng.integers(0, 256, n, dtype=np.uint8)
    wire, _, res = oracle.encode(a, chunk)
    me = oracle.meta_end(n, chunk)
    assert res.wire_len == me + n
    assert _tab(wire, 2, 8).tolist() == [512] * 8
    assert np.array_equal(wire[me:], a)


def test_pack_threshold():
    # S = 253 packs (8256 + 32*253 = 16352 < 16384); S = 254 falls back to RAW
    def tile_with_sum(S):
        E = np.full(8192, 1)
        left = S
        for g in range(32):
            w = min(8, left)
            left -= w
            if w:
                E[g * 256] = 1 + (1 << (w - 1))
        return _bf16_tile(E)
    w253, _, r253 = oracle.encode(tile_with_sum(253), TILE)
    w254, _, r254 = oracle.encode(tile_with_sum(254), TILE)
    assert _tab(w253, 1, 1).tolist() == [511] and r253.payload_bytes == 16352
    assert _tab(w254, 1, 1).tolist() == [512] and r254.payload_bytes == 16384


def _widths_numpy(cache_u8):
    v = cache_u8[: len(cache_u8) // TILE * TILE].view("<u2").astype(np.int64)
    E = ((v >> 7) & 0xFF).reshape(-1, 32, 256)
    rng_ = E.max(axis=2) - E.min(axis=2)
    w = np.where(rng_ > 0, np.floor(np.log2(np.maximum(rng_, 1))).astype(np.int64) + 1, 0)
    return w


def test_size_law_recomputed_with_numpy():
    cfg = inputs.CONFIGS["tiny"]
    a = inputs.make_cache(cfg).numpy()
    wire, _, res = oracle.encode(a, cfg.chunk_bytes)
    S = _widths_numpy(a).sum(axis=1)
    lens = np.where(S <= 253, 8256 + 32 * S, TILE)
    nc, nt = cfg.nbytes // cfg.chunk_bytes, cfg.nbytes // TILE
    assert res.payload_bytes == lens.sum()
    assert _tab(wire, nc, nt).tolist() == np.where(S <= 253, 258 + S, 512).tolist()
    d = _dir(wire, nc)
    per_chunk = lens.reshape(nc, -1).sum(axis=1)
    assert [x[1] for x in d] == per_chunk.tolist()
    assert [x[0] for x in d] == (np.cumsum(per_chunk) - per_chunk).tolist()
    ratio = res.wire_len / cfg.nbytes
    assert 0.70 < ratio < 0.80     # Gaussian bf16: about three quarters


def _worked_example():
    i = np.arange(74228, dtype=np.uint64)
    h = (i * 2654435761) % (1 << 32)
    g, t = i // 256, i // 8192
    m, s = h & 0x7F, (h >> 7) & 1
    E = 118 + ((h >> 8) % (1 + (g % 13)))
    E = np.where(t == 5, (h >> 8) & 0xFF, E)
    v = (s << 15) + (E << 7) + m
    return v.astype("<u2").view(np.uint8)


def _golden():
    out = {}
    for line in open(os.path.join(HERE, "golden", "blueprint_worked_example.txt")):
        line = line.strip()
        if line and not line.startswith("#"):
            k, *v = line.split()
            out[k] = v
    return out


def test_blueprint_worked_example():
    gold = _golden()
    a = _worked_example()
    assert len(a) == 148456
    wire, crc, res = oracle.encode(a, 65536)
    assert [f"{c:08X}" for c in crc] == gold["chunk_crc"]
    assert f"{res.cache_crc:08X}" == gold["cache_crc"][0]
    assert _tab(wire, 3, 10).tolist() == [int(x) for x in gold["tile_tab"]]
    assert oracle.meta_end(len(a), 65536) == int(gold["meta_end"][0])
    assert res.payload_bytes == int(gold["payload_bytes"][0])
    assert res.wire_len == int(gold["wire_len"][0])
    assert f"{_hdr(wire)['meta_crc']:08X}" == gold["meta_crc"][0]
    wire2, crc2, res2 = oracle.encode(a, 65536, dirty=[1, 0, 1], crc_in=crc)
    assert res2.payload_bytes == int(gold["masked_payload_bytes"][0])
    assert res2.wire_len == int(gold["masked_wire_len"][0])
    assert f"{_hdr(wire2)['meta_crc']:08X}" == gold["masked_meta_crc"][0]
    assert _hdr(wire2)["flags"] == 1 and res2.n_present == 2
    # the partial tail tile is stored verbatim at the end of the payload
    assert np.array_equal(wire[-1000:], a[-1000:])
    out, dcrc, r = oracle.decode_verify(wire, len(a), 65536)
    assert r.status == 0 and np.array_equal(out, a) and np.array_equal(dcrc, crc)
    # masked image installs over a destination that already holds chunk 1
    dst = np.zeros_like(a)
    dst[65536:131072] = a[65536:131072]
    out, dcrc, r = oracle.decode_verify(wire2, len(a), 65536, dst=dst, dst_crc=crc)
    assert r.status == 0 and np.array_equal(out, a)
    # ... and is refused when the destination's clean chunk is not the source's
    stale = crc.copy()
    stale[1] ^= 1
    _, _, r = oracle.decode_verify(wire2, len(a), 65536, dst=dst, dst_crc=stale)
    assert (r.status_name, r.first_bad_chunk, r.n_bad_chunks) == ("ERR_STALE", 1, 1)


@pytest.mark.parametrize("name", ["tiny", "engine_small"])
def test_round_trip_configs(name):
    cfg = inputs.CONFIGS[name]
    a = inputs.make_cache(cfg).numpy()
    wire, crc, res = oracle.encode(a, cfg.chunk_bytes)
    assert res.status == 0
    out, dcrc, r = oracle.decode_verify(wire, cfg.nbytes, cfg.chunk_bytes)
    assert r.status == 0 and np.array_equal(out, a) and np.array_equal(dcrc, crc)
    assert np.array_equal(crc, oracle.checksum(a, cfg.chunk_bytes))


def test_round_trip_special_values_and_ragged_sizes():
    rng = np.random.default_rng(4)
    for n in (1, 2, 3, 15, TILE - 1, TILE, TILE + 1, 3 * TILE + 5536, 2 * 65536 + 777):
        a = rng.integers(0, 256, n, dtype=np.uint8)
        if n >= TILE:     # make the first tile compressible, with NaN / Inf / denormal / -0 patterns
            v = rng.integers(0x3E00, 0x4100, 8192).astype("<u2")
            v[:6] = [0x7FC0, 0xFF80, 0x0001, 0x8000, 0x7F80, 0x0000]
            v[256:512] = 0x8000
            a[:TILE] = v.view(np.uint8)
        for chunk in (TILE, 65536):
            wire, crc, res = oracle.encode(a, chunk)
            assert res.status == 0 and res.wire_len <= oracle.wire_bound(n, chunk)
            out, _, r = oracle.decode_verify(wire, n, chunk)
            assert r.status == 0 and np.array_equal(out, a), (n, chunk)


def test_masked_encode_all_clean_is_empty_payload():
    cfg = inputs.CONFIGS["tiny"]
    a = inputs.make_cache(cfg).numpy()
    crc = oracle.checksum(a, cfg.chunk_bytes)
    nc = len(crc)
    wire, crc2, res = oracle.encode(a, cfg.chunk_bytes, dirty=np.zeros(nc, np.uint8), crc_in=crc)
    assert res.payload_bytes == 0 and res.n_present == 0 and res.wire_len == oracle.meta_end(cfg.nbytes, cfg.chunk_bytes)
    assert res.cache_crc == oracle.crc32c(a)
    out, _, r = oracle.decode_verify(wire, cfg.nbytes, cfg.chunk_bytes, dst=a, dst_crc=crc)
    assert r.status == 0 and np.array_equal(out, a)


def test_precopy_round_installs_only_dirty_chunks():
    cfg = inputs.CONFIGS["tiny"]
    prev = inputs.make_cache(cfg)
    cur, rewritten = inputs.rewrite_random_chunks(prev, cfg.chunk_bytes, 0.75, seed=77)
    prev, cur = prev.numpy(), cur.numpy()
    dirty, idx = oracle.dirty_diff(cur, prev, cfg.chunk_bytes)
    assert dirty.tolist() == rewritten.tolist() and dirty.sum() == 24
    crc_prev = oracle.checksum(prev, cfg.chunk_bytes)
    wire, crc_cur, res = oracle.encode(cur, cfg.chunk_bytes, dirty=dirty, crc_in=crc_prev)
    assert res.n_present == 24
    out, dcrc, r = oracle.decode_verify(wire, cfg.nbytes, cfg.chunk_bytes, dst=prev, dst_crc=crc_prev)
    assert r.status == 0 and np.array_equal(out, cur)
    assert np.array_equal(dcrc, oracle.checksum(cur, cfg.chunk_bytes))


def _small_case():
    rng = np.random.default_rng(21)
    n = 2 * TILE + 300
    v = rng.integers(0x3C00, 0x4080, n // 2).astype("<u2")
    a = v.view(np.uint8).copy()
    a[TILE:2 * TILE] = rng.integers(0, 256, TILE, dtype=np.uint8)     # one RAW tile
    return a


def test_every_single_bit_flip_in_metadata_and_descriptors_is_rejected():
    a = _small_case()
    wire, crc, res = oracle.encode(a, TILE)
    me = oracle.meta_end(len(a), TILE)
    assert _tab(wire, 3, 3).tolist()[1:] == [512, 0xFFFF]
    positions = list(range(me * 8)) + list(range(me * 8, (me + 64) * 8))
    for bit in positions:
        w = wire.copy()
        w[bit // 8] ^= 1 << (bit % 8)
        _, dcrc, r = oracle.decode_verify(w, len(a), TILE)
        assert r.status != 0, bit
        assert not dcrc.any()         # the receiver's CRC vector is never updated on failure
        if bit < me * 8:
            assert r.status_name in ("ERR_FORMAT", "ERR_META_CRC"), (bit, r.status_name)
        else:
            assert r.status_name in ("ERR_DESC", "ERR_STRUCT"), (bit, r.status_name)


def test_sampled_payload_bit_flips_are_rejected_by_chunk_crc():
    a = _small_case()
    wire, _, _ = oracle.encode(a, TILE)
    me = oracle.meta_end(len(a), TILE)
    rng = np.random.default_rng(8)
    bits = rng.integers((me + 64) * 8, len(wire) * 8, 600)
    for bit in bits.tolist() + [len(wire) * 8 - 1]:
        w = wire.copy()
        w[bit // 8] ^= 1 << (bit % 8)
        _, _, r = oracle.decode_verify(w, len(a), TILE)
        assert r.status_name == "ERR_CHUNK_CRC" and r.n_bad_chunks == 1, bit


def test_truncation_extension_and_wrong_arguments_are_rejected():
    a = _small_case()
    wire, _, _ = oracle.encode(a, TILE)
    n = len(a)
    assert oracle.decode_verify(wire[:-1], n, TILE)[2].status_name == "ERR_FORMAT"
    assert oracle.decode_verify(np.concatenate([wire, np.zeros(1, np.uint8)]), n, TILE)[2].status_name == "ERR_FORMAT"
    assert oracle.decode_verify(wire[:40], n, TILE)[2].status_name == "ERR_FORMAT"
    assert oracle.decode_verify(wire, n + 2, TILE)[2].status_name == "ERR_FORMAT"
    assert oracle.decode_verify(wire, n, 2 * TILE)[2].status_name == "ERR_FORMAT"


def test_capacity_error_reports_needed_size():
    a = _small_case()
    full, _, res = oracle.encode(a, TILE)
    wire, _, r = oracle.encode(a, TILE, wire_cap=res.wire_len - 1)
    assert r.status_name == "ERR_CAPACITY" and r.wire_len == res.wire_len
    with pytest.raises(ValueError):
        oracle.encode(a, TILE, wire_cap=oracle.meta_end(len(a), TILE) - 1)
    with pytest.raises(ValueError):
        oracle.encode(a, 1000)


# ---------------------------------------------------------------- ZERO tiles (unused allocation)

def _rand_tile(seed):
    rng = np.random.default_rng(seed)
    return (rng.normal(size=8192).astype(np.float32).view(np.uint32) >> 16).astype("<u2").view(np.uint8)


def test_zero_tiles_have_entry_one_and_no_payload():
    a, b = _rand_tile(1), _rand_tile(2)
    z = np.zeros(TILE, dtype=np.uint8)
    cache = np.concatenate([a, z, z, b])
    wire, crc, res = oracle.encode(cache, 4 * TILE, zero_tiles=True)
    wa, _, ra = oracle.encode(a, TILE)
    wb, _, rb = oracle.encode(b, TILE)
    ea, eb = wa[96:ra.wire_len], wb[96:rb.wire_len]
    tab = _tab(wire, 1, 4).tolist()
    assert tab == [int(_tab(wa, 1, 1)[0]), 1, 1, int(_tab(wb, 1, 1)[0])]
    me = oracle.meta_end(4 * TILE, 4 * TILE)
    assert res.payload_bytes == ea.size + eb.size and res.wire_len == me + ea.size + eb.size
    assert np.array_equal(wire[me:me + ea.size], ea) and np.array_equal(wire[me + ea.size:], eb)
    assert _dir(wire, 1)[0][:2] == (0, ea.size + eb.size)
    assert int(crc[0]) == oracle.crc32c(cache)               # the checksum is of the raw bytes, zeros included
    out, dcrc, r = oracle.decode_verify(wire, cache.size, 4 * TILE, dst=np.full(cache.size, 0xEE, np.uint8))
    assert r.status == 0 and np.array_equal(out, cache)


def test_all_zero_cache_is_metadata_plus_its_ragged_tail():
    n = 3 * TILE + 100
    cache = np.zeros(n, dtype=np.uint8)
    wire, crc, res = oracle.encode(cache, 2 * TILE, zero_tiles=True)
    assert _tab(wire, 2, 4).tolist() == [1, 1, 1, 0xFFFF]
    assert res.payload_bytes == 100 and res.wire_len == oracle.meta_end(n, 2 * TILE) + 100
    assert [d[1] for d in _dir(wire, 2)] == [0, 100]
    out, _, r = oracle.decode_verify(wire, n, 2 * TILE, dst=np.full(n, 7, np.uint8))
    assert r.status == 0 and not out.any()


@pytest.mark.parametrize("word", [0x8000, 0x0001, 0x0080])
def test_only_all_zero_bytes_make_a_zero_tile(word):
    # minus zero, the smallest denormal and the smallest normal exponent are data, not emptiness
    tile = np.zeros(8192, dtype="<u2")
    tile[4711] = word
    wire, _, res = oracle.encode(tile.view(np.uint8), TILE, zero_tiles=True)
    assert _tab(wire, 1, 1)[0] >= 258 and res.payload_bytes >= 8256
    out, _, r = oracle.decode_verify(wire, TILE, TILE)
    assert r.status == 0 and np.array_equal(out, tile.view(np.uint8))


def test_constant_tiles_have_entry_two_and_the_value_as_payload():
    """Same option: a tile whose elements all hold one non-zero value (-Inf as a mask fill, 1.0)
    ships as entry 2 and 32 bytes: the value, then zeros.  Written out by hand here."""
    a = _rand_tile(3)
    minus_inf = np.full(8192, 0xFF80, dtype="<u2").view(np.uint8)
    one = np.full(8192, 0x3F80, dtype="<u2").view(np.uint8)
    z = np.zeros(TILE, dtype=np.uint8)
    cache = np.concatenate([minus_inf, a, one, z])
    wire, crc, res = oracle.encode(cache, 2 * TILE, zero_tiles=True)
    wa, _, ra = oracle.encode(a, TILE)
    ea = wa[96:ra.wire_len]
    assert _tab(wire, 2, 4).tolist() == [2, int(_tab(wa, 1, 1)[0]), 2, 1]
    me = oracle.meta_end(4 * TILE, 2 * TILE)
    want = np.concatenate([np.array([0x80, 0xFF] + [0] * 30, np.uint8), ea, np.array([0x80, 0x3F] + [0] * 30, np.uint8)])
    assert np.array_equal(wire[me:], want) and res.payload_bytes == want.size
    assert [d[:2] for d in _dir(wire, 2)] == [(0, 32 + ea.size), (32 + ea.size, 32)]
    assert struct.unpack_from("<H", wire, 6)[0] == 2
    out, dcrc, r = oracle.decode_verify(wire, cache.size, 2 * TILE, dst=np.full(cache.size, 0xEE, np.uint8))
    assert r.status == 0 and np.array_equal(out, cache) and np.array_equal(dcrc, crc)
    # one element off: an ordinary tile again; and without the option nothing changes
    c2 = cache.copy()
    c2[100] ^= 1
    w2, _, _ = oracle.encode(c2, 2 * TILE, zero_tiles=True)
    assert _tab(w2, 2, 4)[0] >= 258
    w3, _, _ = oracle.encode(cache, 2 * TILE)
    assert min(_tab(w3, 2, 4).tolist()) >= 258
    # entry 2 in an image that does not declare the option, a damaged value, a CONST entry on a ragged tile
    bad = wire.copy()
    bad[6] = 0
    assert oracle.decode_verify(_refresh_meta_crc(bad, cache.size, 2 * TILE), cache.size, 2 * TILE)[2].status_name == "ERR_STRUCT"
    bad = wire.copy()
    bad[me] ^= 1
    r = oracle.decode_verify(bad, cache.size, 2 * TILE)[2]
    assert r.status_name == "ERR_CHUNK_CRC" and r.first_bad_chunk == 0
    n = TILE + 64
    rag = np.full(n // 2, 0x3F80, dtype="<u2").view(np.uint8)
    wr, _, _ = oracle.encode(rag, 2 * TILE, zero_tiles=True)
    assert _tab(wr, 1, 2).tolist() == [2, 0xFFFF]
    wr = wr.copy()
    struct.pack_into("<H", wr, 64 + 16 + 2, 2)
    assert oracle.decode_verify(_refresh_meta_crc(wr, n, 2 * TILE), n, 2 * TILE)[2].status_name == "ERR_STRUCT"


def _refresh_meta_crc(wire, nbytes, chunk):
    me = oracle.meta_end(nbytes, chunk)
    w = wire.copy()
    w[52:56] = 0
    w[52:56] = np.frombuffer(struct.pack("<I", oracle.crc32c(w[:me])), dtype=np.uint8)
    return w


def test_zero_entry_is_checked_like_any_other():
    a = _rand_tile(3)
    cache = np.concatenate([a, np.zeros(TILE, np.uint8), a[:500]])
    n, chunk = cache.size, 4 * TILE
    wire, crc, res = oracle.encode(cache, chunk, zero_tiles=True)
    assert _tab(wire, 1, 3).tolist()[1:] == [1, 0xFFFF]
    tab_off = 64 + 16
    # a ZERO entry where a ragged tile belongs: the structure check refuses it
    w = wire.copy(); w[tab_off + 4: tab_off + 6] = (1, 0)
    assert oracle.decode_verify(_refresh_meta_crc(w, n, chunk), n, chunk)[2].status_name == "ERR_STRUCT"
    # a data tile relabelled as ZERO: lengths no longer add up
    w = wire.copy(); w[tab_off: tab_off + 2] = (1, 0)
    assert oracle.decode_verify(_refresh_meta_crc(w, n, chunk), n, chunk)[2].status_name == "ERR_STRUCT"
    # the same with the directory length patched as well: caught by the chunk CRC
    e0 = int(_tab(wire, 1, 3)[0]) * 32
    w[64 + 8: 64 + 12] = np.frombuffer(struct.pack("<I", 500), dtype=np.uint8)
    w = np.concatenate([w[:oracle.meta_end(n, chunk)], w[oracle.meta_end(n, chunk) + e0:]])
    w[32:40] = np.frombuffer(struct.pack("<Q", 500), dtype=np.uint8)
    w[40:48] = np.frombuffer(struct.pack("<Q", w.size), dtype=np.uint8)
    assert oracle.decode_verify(_refresh_meta_crc(w, n, chunk), n, chunk)[2].status_name == "ERR_CHUNK_CRC"
    # without fixing the metadata CRC any of these stops at the metadata check
    w = wire.copy(); w[tab_off + 2] ^= 1
    assert oracle.decode_verify(w, n, chunk)[2].status_name == "ERR_META_CRC"


def test_zero_tiles_are_an_option_recorded_in_the_header():
    cache = np.concatenate([_rand_tile(5), np.zeros(TILE, np.uint8)])
    plain, _, rp = oracle.encode(cache, 2 * TILE)
    opt, _, ro = oracle.encode(cache, 2 * TILE, zero_tiles=True)
    assert _hdr(plain)["flags"] == 0 and _hdr(opt)["flags"] == 2
    assert _tab(plain, 1, 2).tolist()[1] == 258 and _tab(opt, 1, 2).tolist()[1] == 1     # zeros pack to 8256 bytes without it
    assert rp.wire_len - ro.wire_len == 8256
    for w in (plain, opt):
        out, _, r = oracle.decode_verify(w, cache.size, 2 * TILE)
        assert r.status == 0 and np.array_equal(out, cache)
    # entry 1 in an image that does not declare the option is a structure error
    w = opt.copy(); w[6] = 0
    assert oracle.decode_verify(_refresh_meta_crc(w, cache.size, 2 * TILE), cache.size, 2 * TILE)[2].status_name == "ERR_STRUCT"
    # with a dirty mask both flag bits are set
    two = np.concatenate([cache, cache])
    m, _, _ = oracle.encode(two, 2 * TILE, dirty=np.array([1, 0], np.uint8), crc_in=np.zeros(2, np.uint32), zero_tiles=True)
    assert _hdr(m)["flags"] == 3
