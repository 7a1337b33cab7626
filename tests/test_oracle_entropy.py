"""The ENT tile option of the oracle (entropy-coded exponents) against what the format fixes:
hand-built tiles whose streams can be written down without running the coder, the completeness
of the prefix code, Shannon's bound, round trips, and the decoder's verdicts on damaged tiles.
"""
import struct

import numpy as np
import pytest

import oracle

TILE = 16384
META1 = 96            # one chunk of one tile: header 64 + directory 16 + table 2, rounded up to 32

# the code as the format states it: u -> (bits in writing order)
CODE = {0: "00", 1: "10", -1: "01", -2: "1100", 2: "1110", -3: "1101", -4: "11110", -5: "111110", 3: "1111110",
        -6: "11111110"}
ESC = "11111111"


def _tile_of(value_u16):
    return np.full(8192, value_u16, dtype="<u2")


def _encode_one_tile(v):
    # (ent_only: these hand-built tiles are so regular that the bit planes would win the choice)
    wire, crc, res = oracle.encode(v.view(np.uint8), TILE, entropy=True, ent_only=True)
    assert res.status == 0 and oracle.meta_end(TILE, TILE) == META1
    flags = struct.unpack_from("<H", wire, 6)[0]
    entry = struct.unpack_from("<H", wire, 64 + 16)[0]
    return wire, flags, entry, wire[META1:]


def test_prefix_code_is_complete_and_prefix_free():
    words = list(CODE.values()) + [ESC]
    assert sum(2.0 ** -len(w) for w in words) == 1.0                      # Kraft with equality
    for a in words:
        for b in words:
            assert a == b or not b.startswith(a)


def test_constant_tile_by_hand():
    """All elements 1.0 (0x3F80): every anchor is 127, every codeword is '00', a strand is 64 zero
    bits (length byte 0), a share's stream 32 * 64 bits = 64 zero words; the tile is 64 + 8192 + 256
    + 8 * 256 = 10560 bytes = 32 * 330."""
    wire, flags, entry, t = _encode_one_tile(_tile_of(0x3F80))
    assert flags == 4 and entry == (0x8000 | 330) and t.size == 330 * 32
    want = np.zeros(330 * 32, dtype=np.uint8)
    want[0:8] = 127
    want[8:24] = np.full(8, 64, dtype="<u2").view(np.uint8)
    assert np.array_equal(t, want)
    out, _, r = oracle.decode_verify(wire, TILE, TILE)
    assert r.status == 0 and np.array_equal(out.view("<u2"), _tile_of(0x3F80))


def test_one_different_element_lands_where_the_format_says():
    """Share 3, strand 5, element 7 of the strand is 2.0: u = +1, written '10' at bits 14-15 of the
    strand.  Every strand is 64 bits, so strand 5 starts at bit 320 of its share's stream: the set
    bit is bit 334 = word 10, bit 14; share 3's stream starts at word 3 * 64."""
    v = _tile_of(0x3F80)
    elem = 64 * (16 * 3 + 7 // 2) + 2 * 5 + 7 % 2
    v[elem] = 0x4000
    wire, flags, entry, t = _encode_one_tile(v)
    assert entry == (0x8000 | 330)
    assert not t[8256:8512].any()                           # every strand is 64 bits long
    streams = t[8512:].view("<u4")
    want = np.zeros(512, dtype="<u4")
    want[3 * 64 + 10] = 1 << 14
    assert np.array_equal(streams[:512], want)
    assert not t[64:8256].any()                             # sign and mantissa bits are all zero
    out, _, r = oracle.decode_verify(wire, TILE, TILE)
    assert r.status == 0 and np.array_equal(out.view("<u2"), v)


def _escapes_example():
    """Share 0: the first ten elements of strand 0 are 2^20 (E = 147), strand 1 is 0.5 throughout
    (E = 126), everything else 1.0 (E = 127)."""
    v = _tile_of(0x3F80)
    for i in range(10):
        v[64 * (i // 2) + i % 2] = 147 << 7
    for i in range(32):
        v[64 * (i // 2) + 2 + i % 2] = 126 << 7
    return v


def test_strands_follow_one_another_bit_by_bit():
    """The share's exponents add up to 982 * 127 + 10 * 147 + 32 * 126 = 130216, anchor (130216 + 512)
    >> 10 = 127.  Strand 0 is ten escapes (11111111 then E = 147, low bit first: halfword 0x93FF)
    and 22 codewords '00': 204 bits, length byte 140.  Strand 1 starts at bit 204 (word 6, bit 12)
    and codes u = -1 as '01' 32 times: 64 bits of 1010...10 from the high end, byte 0xAA.  The
    share has 204 + 31 * 64 = 2188 bits = 69 words; the tile 8512 + 4 * (69 + 7 * 64) = 10580 bytes,
    rounded up to 10592 = 32 * 331."""
    v = _escapes_example()
    wire, flags, entry, t = _encode_one_tile(v)
    assert list(t[0:8]) == [127] * 8
    assert list(t[8:24].view("<u2")) == [69] + [64] * 7
    assert entry == (0x8000 | 331)
    lens = t[8256:8512]
    assert lens[0] == 140 and not lens[1:].any()
    s = t[8512:].view("<u4")
    want = np.zeros(s.size, dtype="<u4")
    want[0:5] = 0x93FF93FF
    want[6], want[7], want[8] = 0xAAAAA000, 0xAAAAAAAA, 0x00000AAA
    assert np.array_equal(s, want)
    out, _, r = oracle.decode_verify(wire, TILE, TILE)
    assert r.status == 0 and np.array_equal(out.view("<u2"), v)


def test_a_strand_too_long_for_its_length_byte_keeps_the_tile_out_of_the_form():
    """A strand of 32 escapes would be 512 bits; the length byte ends at 319.  Such a tile is stored
    in one of the other forms (here raw under ent_only, PACK otherwise), and 319 bits still fit."""
    v = _tile_of(0x3F80)
    for i in range(32):
        v[64 * (i // 2) + i % 2] = 147 << 7
    wire, flags, entry, t = _encode_one_tile(v)
    assert entry == 512
    w2, _, _ = oracle.encode(v.view(np.uint8), TILE, entropy=True)
    assert 258 <= struct.unpack_from("<H", w2, 64 + 16)[0] < 512
    # 18 escapes, one 5-bit codeword (u = -4) and 13 codewords of 2 bits: 288 + 5 + 26 = 319 bits
    v = _tile_of(0x3F80)
    for i in range(18):
        v[64 * (i // 2) + i % 2] = 147 << 7
    v[64 * 9] = 123 << 7
    wire, flags, entry, t = _encode_one_tile(v)
    assert entry & 0x8000 and t[8256] == 255
    out, _, r = oracle.decode_verify(wire, TILE, TILE)
    assert r.status == 0 and np.array_equal(out.view("<u2"), v)


def _gauss(n, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    return ((rng.normal(size=n) * scale).astype(np.float32).view(np.uint32) >> 16).astype("<u2")


def _strand_view(v):
    """exponents as [tile, share, row, strand, half] -> [tile, share, strand, i]"""
    E = ((v >> 7) & 0xFF).astype(np.int64).reshape(-1, 8, 16, 32, 2)
    return E.transpose(0, 1, 3, 2, 4).reshape(E.shape[0], 8, 32, 32)


def test_sizes_follow_the_code_lengths_and_respect_shannon():
    v = np.concatenate([_gauss(8192 * 3, 5), _gauss(8192 * 2, 6, 37.0), _gauss(8192, 7, 1e-3)])
    n_tiles = v.size // 8192
    wire, crc, res = oracle.encode(v.view(np.uint8), 2 * TILE, entropy=True)
    me = oracle.meta_end(v.size * 2, 2 * TILE)
    entries = wire[64 + 16 * 3: 64 + 16 * 3 + 2 * n_tiles].view("<u2")
    E = _strand_view(v)
    anchor = (E.sum(axis=(2, 3)) + 512) >> 10
    u = E - anchor[:, :, None, None]
    L = np.full(u.shape, 16)
    for k, w in CODE.items():
        L[u == k] = len(w)
    strand_bits = L.sum(axis=3)                                           # [tile, share, strand]
    words = -(-strand_bits.sum(axis=2) // 32)
    want_len = (8512 + 4 * words.sum(axis=1) + 31) // 32 * 32
    want_len = np.where(strand_bits.max(axis=(1, 2)) > 319, TILE, want_len)  # a strand the length byte cannot hold
    # the bit-plane form of the same tiles: 32 groups of 256 elements in memory order
    G = ((v >> 7) & 0xFF).astype(np.int64).reshape(n_tiles, 32, 256)
    rng_ = G.max(axis=2) - G.min(axis=2)
    S = np.where(rng_ > 0, np.floor(np.log2(np.maximum(rng_, 1))).astype(np.int64) + 1, 0).sum(axis=1)
    pack_len = np.where(S <= 253, 8256 + 32 * S, TILE)
    best = np.minimum(np.minimum(want_len, pack_len), TILE)
    want_entry = np.where(want_len < pack_len, 0x8000 | (want_len // 32), np.where(S <= 253, 258 + S, 512))
    assert np.array_equal(entries.astype(np.int64), want_entry)
    assert res.wire_len == me + int(best.sum())
    assert (entries & 0x8000).any()                           # the Gaussian tiles do take the ENT form
    only, _, res_only = oracle.encode(v.view(np.uint8), 2 * TILE, entropy=True, ent_only=True)
    assert res_only.wire_len == me + int(np.minimum(want_len, TILE).sum())
    # no uniquely decodable code beats the empirical entropy of what it codes
    for t in range(n_tiles):
        for s in range(8):
            c = np.bincount(E[t, s].ravel(), minlength=256).astype(float)
            p = c[c > 0] / 1024.0
            assert L[t, s].sum() >= 1024.0 * -(p * np.log2(p)).sum() - 1e-6
    # and on Gaussian data it stays within half a bit of it on average, far below the plane packing
    w_pack, _, r_pack = oracle.encode(v.view(np.uint8), 2 * TILE)
    assert res.wire_len < 0.93 * r_pack.wire_len


@pytest.mark.parametrize("n,chunk", [(5 * TILE + 300, 2 * TILE), (4 * TILE, 4 * TILE), (TILE - 2, TILE), (9 * TILE + 1, 4 * TILE)])
def test_round_trip_masks_and_special_values(n, chunk):
    rng = np.random.default_rng(n)
    a = _gauss((n + 1) // 2, n).view(np.uint8)[:n].copy()
    if n >= 2 * TILE:
        a[TILE:2 * TILE] = rng.integers(0, 256, TILE, dtype=np.uint8)       # incompressible: stays raw
        sp = a[:TILE].view("<u2")
        sp[:6] = [0x7FC0, 0xFF80, 0x0001, 0x8000, 0x7F80, 0x0000]           # NaN, -Inf, denormal, -0, Inf, 0
    nc = oracle.num_chunks(n, chunk)
    wire, crc, res = oracle.encode(a, chunk, entropy=True)
    assert res.status == 0 and np.array_equal(crc, oracle.checksum(a, chunk))
    out, dcrc, r = oracle.decode_verify(wire, n, chunk)
    assert r.status == 0 and np.array_equal(out, a) and np.array_equal(dcrc, crc)
    if n >= 2 * TILE:
        entries = wire[64 + 16 * nc: 64 + 16 * nc + 4].view("<u2")
        assert entries[1] == 512 and entries[0] & 0x8000
    # with a mask: absent chunks are trusted, the rest is coded the same way
    dirty = (np.arange(nc) % 2 == 0).astype(np.uint8)
    wire2, crc2, res2 = oracle.encode(a, chunk, dirty=dirty, crc_in=crc, entropy=True)
    base = a.copy()
    out2, _, r2 = oracle.decode_verify(wire2, n, chunk, dst=base, dst_crc=crc)
    assert res2.status == 0 and r2.status == 0 and np.array_equal(out2, a)
    assert struct.unpack_from("<H", wire2, 6)[0] == 5
    # both options together: a zero tile is an entry, the rest ENT
    if n >= 3 * TILE:
        z = a.copy()
        z[2 * TILE:3 * TILE] = 0
        wz, _, rz = oracle.encode(z, chunk, zero_tiles=True, entropy=True)
        oz, _, rdz = oracle.decode_verify(wz, n, chunk)
        assert rz.status == 0 and rdz.status == 0 and np.array_equal(oz, z)
        assert struct.unpack_from("<H", wz, 64 + 16 * nc + 4)[0] == 1 and struct.unpack_from("<H", wz, 6)[0] == 6


def _reseal(w, n, chunk):
    me = oracle.meta_end(n, chunk)
    z = w[:me].copy()
    z[52:56] = 0
    w[52:56] = np.frombuffer(struct.pack("<I", oracle.crc32c(z)), dtype=np.uint8)
    return w


def test_damaged_ent_tiles_are_refused_with_the_right_status():
    n, chunk = 4 * TILE, 2 * TILE
    a = _gauss(n // 2, 21).view(np.uint8)
    wire, crc, res = oracle.encode(a, chunk, entropy=True)
    me = oracle.meta_end(n, chunk)
    entries = wire[64 + 16 * 2: 64 + 16 * 2 + 8].view("<u2")
    len0 = 32 * int(entries[0] & 0x7FFF)
    # a count that no longer adds up to the entry: structure
    w = wire.copy()
    w[me + 8] ^= 16                       # 16 halfwords = one 32-byte unit
    assert oracle.decode_verify(w, n, chunk)[2].status_name == "ERR_STRUCT"
    # counts moved between shares (sum unchanged): the streams are no longer used up exactly
    w = wire.copy()
    c = w[me + 8: me + 24].view("<u2")
    c[0] += 1
    c[1] -= 1
    r = oracle.decode_verify(w, n, chunk)[2]
    assert r.status_name == "ERR_DESC" and r.first_bad_chunk == 0 and r.n_bad_chunks == 1
    # in the second tile of the second chunk: lowest failing tile decides, chunk 1 is reported
    w = wire.copy()
    off = me + len0 + 32 * int(entries[1] & 0x7FFF) + 32 * int(entries[2] & 0x7FFF)
    c = w[off + 8: off + 24].view("<u2")
    c[6] += 2
    c[7] -= 2
    r = oracle.decode_verify(w, n, chunk)[2]
    assert r.status_name == "ERR_DESC" and r.first_bad_chunk == 1
    # a flipped bit inside a stream: either the streams no longer fit (DESC) or the bytes differ (CHUNK_CRC)
    seen = set()
    for k in range(0, 600, 7):
        w = wire.copy()
        w[me + 8256 + k] ^= 1 << (k % 8)
        seen.add(oracle.decode_verify(w, n, chunk)[2].status_name)
    assert seen <= {"ERR_DESC", "ERR_CHUNK_CRC"} and "ERR_CHUNK_CRC" in seen
    # an ENT entry in an image that does not declare the option
    w = wire.copy()
    w[6] = 0
    assert oracle.decode_verify(_reseal(w, n, chunk), n, chunk)[2].status_name == "ERR_STRUCT"
    # a PACK tile is at home in an image that declares the option (the encoder picks the shorter form)
    wp, _, _ = oracle.encode(a, chunk)
    wp = wp.copy()
    wp[6] = 4
    out_p, _, r_p = oracle.decode_verify(_reseal(wp, n, chunk), n, chunk)
    assert r_p.status == 0 and np.array_equal(out_p, a)
    # flags above 7 are no format this decoder knows
    w = wire.copy()
    w[6] = 12
    assert oracle.decode_verify(_reseal(w, n, chunk), n, chunk)[2].status_name == "ERR_FORMAT"


def test_default_images_are_unchanged_by_the_option():
    a = _gauss(3 * 8192, 31).view(np.uint8)
    w0, _, r0 = oracle.encode(a, TILE)
    assert struct.unpack_from("<H", w0, 6)[0] == 0 and not (w0[64 + 48: 64 + 48 + 6].view("<u2") & 0x8000).any()


def test_every_codeword_bit_by_bit():
    """Share 0, strand 0 starts with one element for each coded u (in the table's order), all else
    is E = 127.  The strand's bit string is the codewords as the format lists them, 44 bits, then 22
    times '00': 88 bits, length byte 24; it is the head of the share's stream, the other strands
    (64 zero bits each) follow: 88 + 31 * 64 = 2072 bits = 65 words."""
    us = [0, 1, -1, -2, 2, -3, -4, -5, 3, -6]
    v = _tile_of(0x3F80)
    for i, u in enumerate(us):
        v[64 * (i // 2) + i % 2] = (127 + u) << 7
    wire, flags, entry, t = _encode_one_tile(v)
    assert t[0] == 127
    bits = "".join(CODE[u] for u in us) + "00" * 22
    assert len(bits) == 88
    bits += "0" * 8
    words = [sum(int(bits[32 * k + b]) << b for b in range(32)) for k in range(3)]
    s = t[8512:].view("<u4")
    assert struct.unpack_from("<H", t, 8)[0] == 65 and t[8256] == 24 and not t[8257:8512].any()
    assert [int(x) for x in s[:3]] == words and not s[3:].any()
    out, _, r = oracle.decode_verify(wire, TILE, TILE)
    assert r.status == 0 and np.array_equal(out.view("<u2"), v)


def test_the_option_never_makes_an_image_longer():
    """Per tile the shortest of ENT, PACK and raw is stored (PACK on a tie): regular data, where
    the bit planes cost next to nothing, keeps its PACK tiles; an image with the option is never
    longer than one without."""
    const = _tile_of(0x3F80)                                              # one exponent: PACK at 8256 bytes
    narrow = ((np.arange(8192) % 2 + 126) << 7).astype("<u2")             # two exponents everywhere: width 1
    gauss = _gauss(8192, 77)
    noise = np.random.default_rng(5).integers(0, 65536, 8192).astype("<u2")
    v = np.concatenate([const, narrow, gauss, noise])
    w_opt, _, r_opt = oracle.encode(v.view(np.uint8), 4 * TILE, entropy=True)
    w_def, _, r_def = oracle.encode(v.view(np.uint8), 4 * TILE)
    e_opt = w_opt[64 + 16: 64 + 16 + 8].view("<u2")
    e_def = w_def[64 + 16: 64 + 16 + 8].view("<u2")
    assert list(e_opt[:2]) == list(e_def[:2]) == [258, 258 + 32]          # PACK kept
    assert e_opt[2] & 0x8000 and 258 <= e_def[2] < 512                    # ENT wins on the Gaussian tile
    assert e_opt[3] == e_def[3] == 512                                    # noise stays raw
    assert r_opt.wire_len < r_def.wire_len
    out, _, r = oracle.decode_verify(w_opt, v.size * 2, 4 * TILE)
    assert r.status == 0 and np.array_equal(out, v.view(np.uint8))
    for seed in range(6):
        x = _gauss(8192 * 3, 100 + seed, float(2.0 ** (seed - 3)))
        x[:8192] = (x[:8192] & 0x807F) | (120 << 7)                        # a tile with one exponent
        a_, _, ra = oracle.encode(x.view(np.uint8), TILE, entropy=True)
        b_, _, rb = oracle.encode(x.view(np.uint8), TILE)
        ea, eb = a_[64 + 48: 64 + 48 + 6].view("<u2"), b_[64 + 48: 64 + 48 + 6].view("<u2")
        la = np.where(ea & 0x8000, 32 * (ea & 0x7FFF).astype(np.int64), 32 * ea.astype(np.int64))
        assert (la <= 32 * eb.astype(np.int64)).all() and ra.wire_len <= rb.wire_len


def _golden():
    import os
    ex = {}
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "ent_worked_examples.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, key, *rest = line.split()
        ex.setdefault(name, {}).setdefault(key, []).append(rest)
    return ex


def test_golden_worked_examples():
    """The fixtures were written down from the format statement before looking at the coder's output."""
    ex = _golden()
    for name, spec in ex.items():
        v = _tile_of(0x3F80)
        if name == "one_odd":
            e = spec["element"][0]
            v[int(e[0])] = int(e[2], 16)
        if name == "escapes":
            v = _escapes_example()
        wire, flags, entry, t = _encode_one_tile(v)
        if "anchors" in spec:
            assert list(t[0:8]) == [int(x) for x in spec["anchors"][0]], name
        if "counts" in spec:
            assert list(t[8:24].view("<u2")) == [int(x) for x in spec["counts"][0]], name
        if "entry" in spec:
            assert entry == int(spec["entry"][0][0], 16), name
        lens = np.zeros(256, dtype=np.int64)
        for item in spec.get("lengths", [[]])[0]:
            at, val = item.split(":")
            lens[int(at)] = int(val)
        assert list(t[8256:8512]) == list(lens), name
        counts = t[8:24].view("<u2")
        for sh in spec.get("share", []):
            share = int(sh[0])
            start = int(counts[:share].sum())
            stream = t[8512 + 4 * start: 8512 + 4 * (start + int(counts[share]))].view("<u4")
            want = np.zeros(stream.size, dtype=np.int64)
            for item in sh[2:]:
                rng_, val = item.split(":")
                lo, hi = (rng_.split("-") + [rng_])[:2]
                want[int(lo): int(hi) + 1] = int(val, 16)
            assert [int(x) for x in stream] == list(want), name
        listed = {int(sh[0]) for sh in spec.get("share", [])}
        for share in range(8):
            if share not in listed:
                start = int(counts[:share].sum())
                assert not t[8512 + 4 * start: 8512 + 4 * (start + int(counts[share]))].any(), (name, share)


def test_no_bit_of_an_image_with_both_options_can_flip_unnoticed():
    """Every single bit of a small image that holds an ENT tile, a CONST tile, a ZERO tile and a
    ragged tail (zero-tile and entropy options together): flipped, the image is refused.  That
    includes the bytes that carry no data: the spare bytes of an ENT tile's header, the fill behind
    its last stream, the zeros behind a CONST tile's value; and the anchors, which must be the
    rounded means of what their shares decode to."""
    a = np.concatenate([_gauss(TILE // 2, 31).view(np.uint8), np.full(8192, 0xFF80, "<u2").view(np.uint8),
                        np.zeros(TILE, np.uint8), _gauss(150, 32).view(np.uint8)])
    n, chunk = a.size, 4 * TILE
    wire, crc, res = oracle.encode(a, chunk, zero_tiles=True, entropy=True)
    nt = oracle.num_tiles(n)
    tab = wire[64 + 16: 64 + 16 + 2 * nt].view(np.uint16).tolist()
    assert tab[0] & 0x8000 and tab[0] != 0xFFFF and tab[1:] == [2, 1, 0xFFFF]
    out, _, r = oracle.decode_verify(wire, n, chunk, expect_entropy=True)
    assert r.status == 0 and np.array_equal(out, a)
    accepted = []
    for bit in range(wire.size * 8):
        w = wire.copy()
        w[bit // 8] ^= 1 << (bit % 8)
        if oracle.decode_verify(w, n, chunk, expect_entropy=True)[2].status == 0:
            accepted.append(bit)
    assert not accepted, f"{len(accepted)} flipped bits were accepted, first at byte {accepted[0] // 8}"


def test_spare_bytes_and_anchors_of_coded_tiles_are_checked():
    v = _gauss(TILE // 2, 33)
    wire, _, res = oracle.encode(v.view(np.uint8), TILE, entropy=True)
    me = oracle.meta_end(TILE, TILE)
    words = int(wire[me + 8: me + 24].view(np.uint16).astype(np.int64).sum())
    spots = [me + 24, me + 63]                               # spare header bytes
    if 8512 + 4 * words < res.wire_len - me:
        spots.append(res.wire_len - 1)                       # the last fill byte, when the tile has fill
    for at in spots:
        w = wire.copy()
        w[at] ^= 0x40
        assert oracle.decode_verify(w, TILE, TILE)[2].status_name == "ERR_DESC", at
    # an anchor that moves shifts everything its share decodes to, which the chunk CRC sees
    w = wire.copy()
    w[me + 3] += 1
    assert oracle.decode_verify(w, TILE, TILE)[2].status_name == "ERR_CHUNK_CRC"
    # ... but the same exponents can be written with another anchor: E = 127 everywhere is '00' under
    # anchor 127 and '10' (u = +1) under anchor 126.  Such an image decodes to the right bytes; it is
    # refused because an anchor must be the rounded mean of what its share decodes to.
    wire, _, res = oracle.encode(_tile_of(0x3F80).view(np.uint8), TILE, entropy=True, ent_only=True)
    assert oracle.decode_verify(wire, TILE, TILE)[2].status == 0
    w = wire.copy()
    w[me + 0] = 126
    w[me + 8512: me + 8512 + 256] = 0x55                     # '10' is the number 1 in a 2-bit field
    assert oracle.decode_verify(w, TILE, TILE)[2].status_name == "ERR_DESC"
    # a strand length that does not match its codewords
    w = wire.copy()
    w[me + 8256 + 7] = 2
    assert oracle.decode_verify(w, TILE, TILE)[2].status_name == "ERR_DESC"
