"""Seeded random damage (bit flips, byte overwrites, truncation) anywhere in a wire image, for every
option set: the GPU's verdict (status, first bad chunk, count) must be the oracle's, and a refused
image must leave the destination's checksums alone."""
import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu
TILE = 16384


def _image(option, seed):
    rng = np.random.default_rng(seed)
    chunk = int(rng.choice([1, 2, 4])) * TILE
    n = int(rng.integers(2, 12)) * TILE + int(rng.integers(0, 2)) * int(rng.integers(1, TILE))
    v = (rng.normal(size=(n + 1) // 2) * float(2.0 ** rng.integers(-3, 4))).astype(np.float32)
    a = (v.view(np.uint32) >> 16).astype("<u2").view(np.uint8)[:n].copy()
    nt = n // TILE
    if nt > 2:
        a[TILE:2 * TILE] = 0                                        # a zero tile
        a[2 * TILE:3 * TILE].view("<u2")[:] = 0x3F80 + int(rng.integers(0, 2))     # a constant tile
    if nt > 4:
        a[4 * TILE:5 * TILE] = rng.integers(0, 256, TILE, dtype=np.uint8)          # a raw tile
    wire, crc, res = oracle.encode(a, chunk, zero_tiles="zero" in option, entropy="entropy" in option)
    return a, n, chunk, wire, crc


def damage(wire, n, chunk, rng):
    w = wire.copy()
    me = oracle.meta_end(n, chunk)
    kind = rng.integers(0, 8)
    if kind == 0:                                   # a bit anywhere
        i = int(rng.integers(0, w.size)); w[i] ^= 1 << int(rng.integers(0, 8))
    elif kind == 1:                                 # a bit in the metadata
        i = int(rng.integers(0, me)); w[i] ^= 1 << int(rng.integers(0, 8))
    elif kind == 2:                                 # a bit near the start of some tile's payload (descriptors, counts)
        i = me + int(rng.integers(0, max(1, (w.size - me) // 64))) * 64 + int(rng.integers(0, 64))
        i = min(i, w.size - 1); w[i] ^= 1 << int(rng.integers(0, 8))
    elif kind == 3:                                 # a run of bytes overwritten
        i = int(rng.integers(me, w.size)); k = int(rng.integers(1, 200))
        w[i:i + k] = rng.integers(0, 256, min(k, w.size - i), dtype=np.uint8)
    elif kind == 4:                                 # a table entry replaced, metadata CRC made right again
        import struct
        nc = oracle.num_chunks(n, chunk)
        t = int(rng.integers(0, oracle.num_tiles(n)))
        struct.pack_into("<H", w, 64 + 16 * nc + 2 * t, int(rng.choice([0, 1, 2, 258, 300, 512, 0x8000 | 300, 0x8000 | 511, 0xFFFF, 7])))
        z = w[:me].copy(); z[52:56] = 0
        w[52:56] = np.frombuffer(struct.pack("<I", oracle.crc32c(z)), dtype=np.uint8)
    elif kind in (5, 6):                            # a directory field altered (an offset, or a length: every later
        import struct                               # chunk is then off the running sum), metadata CRC made right again
        c = int(rng.integers(0, oracle.num_chunks(n, chunk)))
        if kind == 5:
            po = struct.unpack_from("<Q", w, 64 + 16 * c)[0]
            struct.pack_into("<Q", w, 64 + 16 * c, po + 32 * int(rng.integers(1, 5)))
        else:
            el = struct.unpack_from("<I", w, 64 + 16 * c + 8)[0]
            struct.pack_into("<I", w, 64 + 16 * c + 8, max(0, el + 32 * int(rng.integers(-2, 3))))
        z = w[:me].copy(); z[52:56] = 0
        w[52:56] = np.frombuffer(struct.pack("<I", oracle.crc32c(z)), dtype=np.uint8)
    else:                                           # truncated or extended
        k = int(rng.integers(1, 100))
        w = w[:-k].copy() if rng.integers(0, 2) else np.concatenate([w, np.zeros(k, np.uint8)])
    return w


@pytest.mark.parametrize("option", ["default", "zero", "entropy", "zero+entropy"])
@pytest.mark.parametrize("seed", range(4))
def test_damaged_images_get_the_oracles_verdict(option, seed):
    import torch
    from paper_2607_10389_b200 import binding as wm
    a, n, chunk, wire, crc = _image(option, 7000 + seed)
    ent = "entropy" in option
    nc = oracle.num_chunks(n, chunk)
    ws = wm.new_workspace(n, chunk)
    res = wm.new_result()
    rng = np.random.default_rng(9000 + seed)
    live_crc = np.arange(nc, dtype=np.uint32) + 5
    seen = set()
    for k in range(40):
        w = damage(wire, n, chunk, rng)
        want = oracle.decode_verify(w, n, chunk, dst=np.zeros(n, np.uint8), dst_crc=live_crc, expect_entropy=ent)[2]
        pad = (-w.size) % 16
        dev = torch.from_numpy(np.concatenate([w, np.zeros(pad, np.uint8)])).cuda()
        dst = torch.zeros(n, dtype=torch.uint8, device="cuda")
        dcrc = torch.from_numpy(live_crc.view(np.int32).copy()).cuda()
        strict = wm.OPT_STRICT if k % 2 else 0
        wm.wm_decode_verify_opt(dev, w.size, dst, chunk, dcrc, ws, res, (wm.OPT_ENTROPY if ent else 0) | strict)
        r = wm.read_result(res)
        assert (r.status, r.first_bad_chunk, r.n_bad_chunks) == (want.status, want.first_bad_chunk, want.n_bad_chunks), \
            (option, seed, k, r.status_name, want.status_name)
        got_crc = dcrc.cpu().numpy().view(np.uint32)
        if want.status != 0:
            assert np.array_equal(got_crc, live_crc)
            if strict:
                assert not bool(dst.any())
        else:                                       # damage where nothing looks (fill bytes): still the cache
            assert np.array_equal(dst.cpu().numpy(), a) and np.array_equal(got_crc, crc)
        seen.add(want.status_name)
    assert len(seen) >= 3
