"""wm_decode_verify_strict: nothing is stored until every check has passed."""
import struct

import numpy as np
import pytest

import oracle

TILE = 16384


def _cache(n, seed):
    rng = np.random.default_rng(seed)
    return (rng.normal(size=(n + 1) // 2).astype(np.float32).view(np.uint32) >> 16).astype("<u2").view(np.uint8)[:n].copy()


def test_oracle_strict_leaves_the_destination_alone_on_failure():
    n, chunk = 5 * TILE + 300, 2 * TILE
    a = _cache(n, 1)
    wire, crc, res = oracle.encode(a, chunk)
    live = np.full(n, 0x42, dtype=np.uint8)
    live_crc = np.arange(crc.size, dtype=np.uint32)
    out, dcrc, r = oracle.decode_verify_strict(wire, n, chunk, live, live_crc)
    assert r.status == 0 and np.array_equal(out, a) and np.array_equal(dcrc, crc)
    bad = wire.copy()
    bad[-7] ^= 2
    out, dcrc, r = oracle.decode_verify_strict(bad, n, chunk, live, live_crc)
    assert r.status_name == "ERR_CHUNK_CRC" and np.array_equal(out, live) and np.array_equal(dcrc, live_crc)


def _damage(wire, n, chunk, kind):
    """Damaged copies of a good image, one per kind of failure after the metadata checks."""
    me = oracle.meta_end(n, chunk)
    w = wire.copy()
    if kind == "payload":
        w[me + 9000] ^= 0x40
    elif kind == "last_byte":
        w[-1] ^= 1
    elif kind == "descriptor":
        w[me + 3] ^= 0x10                     # check nibble of a group descriptor
    elif kind == "meta":
        w[70] ^= 1
    elif kind == "truncated":
        w = w[:-32]
    elif kind == "cache_crc":
        w[48] ^= 1
        z = w[:me].copy(); z[52:56] = 0
        w[52:56] = np.frombuffer(struct.pack("<I", oracle.crc32c(z)), dtype=np.uint8)
    return w


@pytest.mark.gpu
@pytest.mark.parametrize("n,chunk", [(9 * TILE + 1234, 4 * TILE), (6 * TILE, 2 * TILE), (2 * TILE + 3, TILE)])
def test_strict_decode_matches_the_oracle_and_writes_only_on_success(n, chunk):
    import torch
    from paper_2607_10389_b200 import binding as wm
    a = _cache(n, n % 97)
    nc = wm.num_chunks(n, chunk)
    dirty = (np.arange(nc) % 3 != 0).astype(np.uint8)
    dirty[-1] = 1
    crc_prev = np.full(nc, 0xABCD0123, dtype=np.uint32)
    ws, res = wm.new_workspace(n, chunk), wm.new_result()
    for d_np in (None, dirty):
        wire_np, crc_np, r_enc = oracle.encode(a, chunk, dirty=d_np, crc_in=crc_prev)
        assert r_enc.status == 0
        live = np.full(n, 0x5C, dtype=np.uint8)
        live_crc = crc_prev.copy()
        for kind in ("good", "payload", "last_byte", "descriptor", "meta", "truncated", "cache_crc"):
            w_np = wire_np if kind == "good" else _damage(wire_np, n, chunk, kind)
            want_out, want_crc, want = oracle.decode_verify_strict(w_np, n, chunk, live, live_crc)
            wire = torch.from_numpy(np.concatenate([w_np, np.zeros((-w_np.size) % 16 + 16, np.uint8)])).cuda()
            dst = torch.from_numpy(live.copy()).cuda()
            dcrc = torch.from_numpy(live_crc.view(np.int32).copy()).cuda()
            wm.wm_decode_verify_strict(wire, w_np.size, dst, chunk, dcrc, ws, res)
            r = wm.read_result(res)
            assert r.status == want.status, (kind, r.status_name, want.status_name)
            assert (r.first_bad_chunk, r.n_bad_chunks) == (want.first_bad_chunk, want.n_bad_chunks)
            assert np.array_equal(dst.cpu().numpy(), want_out), kind
            assert np.array_equal(dcrc.cpu().numpy().view(np.uint32), want_crc), kind
            if kind == "good":
                assert r.ok
                if d_np is None:
                    assert np.array_equal(want_out, a)
            else:
                assert not r.ok and np.array_equal(dst.cpu().numpy(), live)       # not one byte stored
            # the ordinary call agrees on the verdict
            dst2 = torch.from_numpy(live.copy()).cuda()
            dcrc2 = torch.from_numpy(live_crc.view(np.int32).copy()).cuda()
            wm.wm_decode_verify(wire, w_np.size, dst2, chunk, dcrc2, ws, res)
            assert wm.read_result(res).status == want.status
