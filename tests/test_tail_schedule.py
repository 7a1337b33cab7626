"""Verification placement: the move cut into super-chunks on three streams (encode, wire copy,
decode + verify).  Every part is a wire image of its own and must equal the oracle's image of
that byte range; a part damaged on the wire fails alone.
"""
import numpy as np
import pytest

import oracle

TILE = 16384


def test_plan_covers_the_cache_once_and_keeps_chunks_whole():
    from paper_2607_10389_b200 import tail_schedule as ts
    try:
        parts = ts.plan_parts(10 * 65536 + 77, 65536, 4 * 65536)
    except ts.wm.WmError:
        pytest.skip("library not built")
    assert [p.nbytes for p in parts] == [4 * 65536, 4 * 65536, 2 * 65536 + 77]
    assert [p.offset for p in parts] == [0, 4 * 65536, 8 * 65536]
    assert [p.first_chunk for p in parts] == [0, 4, 8] and [p.n_chunks for p in parts] == [4, 4, 3]
    for a, b in zip(parts, parts[1:]):
        assert b.wire_offset >= a.wire_offset + a.wire_cap and b.wire_offset % 16 == 0
    for p in parts:
        assert p.wire_cap == oracle.wire_bound(p.nbytes, 65536)
    with pytest.raises(ts.wm.WmError):
        ts.plan_parts(1 << 20, 65536, 3 * 65536 + 1)
    with pytest.raises(ts.wm.WmError):
        ts.plan_parts(0, 65536, 65536)


def _cache(n, seed):
    rng = np.random.default_rng(seed)
    return (rng.normal(size=(n + 1) // 2).astype(np.float32).view(np.uint32) >> 16).astype("<u2").view(np.uint8)[:n].copy()


@pytest.mark.gpu
@pytest.mark.parametrize("strict,entropy", [(False, False), (True, False), (False, True), (True, True)])
def test_every_part_is_the_oracles_image_of_its_range(strict, entropy):
    import torch
    from paper_2607_10389_b200 import tail_schedule as ts
    chunk, sup = 4 * TILE, 12 * TILE
    n = 3 * sup + 5 * TILE + 321                         # three full parts and a ragged one
    a = _cache(n, 11)
    sched = ts.TailSchedule(n, chunk, sup, strict=strict, entropy=entropy)
    assert len(sched.parts) == 4
    nc = oracle.num_chunks(n, chunk)
    src = torch.from_numpy(a).cuda()
    dst = torch.full((n,), 0x5A, dtype=torch.uint8, device="cuda")
    src_crc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    dst_crc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    rep = sched.move(src, dst, src_crc, dst_crc)
    assert rep.ok and rep.total_ms > 0 and rep.exposed_ms > 0 and sched.launches > 0
    assert np.array_equal(dst.cpu().numpy(), a)
    want_crc = oracle.checksum(a, chunk)
    assert np.array_equal(src_crc.cpu().numpy().view(np.uint32), want_crc)
    assert np.array_equal(dst_crc.cpu().numpy().view(np.uint32), want_crc)
    total = 0
    for p, re, rd in zip(sched.parts, rep.encode, rep.decode):
        wire, crc, res = oracle.encode(a[p.offset: p.offset + p.nbytes], chunk, entropy=entropy)
        assert re.wire_len == wire.size == res.wire_len and re.cache_crc == res.cache_crc == rd.cache_crc
        got = sched.wire_recv[p.wire_offset: p.wire_offset + re.wire_len].cpu().numpy()
        assert np.array_equal(got, wire)
        assert rd.n_present == p.n_chunks
        total += wire.size
    assert rep.wire_bytes == total


@pytest.mark.gpu
@pytest.mark.parametrize("strict", [False, True])
def test_a_part_damaged_on_the_wire_fails_alone(strict):
    import torch
    from paper_2607_10389_b200 import tail_schedule as ts
    chunk, sup = 2 * TILE, 8 * TILE
    n = 4 * sup
    a = _cache(n, 12)
    sched = ts.TailSchedule(n, chunk, sup, strict=strict)
    nc = oracle.num_chunks(n, chunk)
    src = torch.from_numpy(a).cuda()
    dst = torch.full((n,), 0x5A, dtype=torch.uint8, device="cuda")
    src_crc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    dst_crc = torch.full((nc,), 99, dtype=torch.int32, device="cuda")

    def tamper(part, image):
        if part.index == 2:
            image[image.numel() - 5] ^= 8

    rep = sched.move(src, dst, src_crc, dst_crc, tamper=tamper)
    assert [r.ok for r in rep.encode] == [True] * 4
    assert [r.status_name for r in rep.decode] == ["OK", "OK", "ERR_CHUNK_CRC", "OK"]
    bad = sched.parts[2]
    assert rep.decode[2].first_bad_chunk == bad.n_chunks - 1 and rep.decode[2].n_bad_chunks == 1
    want_crc = oracle.checksum(a, chunk)
    got_crc = dst_crc.cpu().numpy().view(np.uint32)
    out = dst.cpu().numpy()
    for p in sched.parts:
        ck = slice(p.first_chunk, p.first_chunk + p.n_chunks)
        by = slice(p.offset, p.offset + p.nbytes)
        if p.index == 2:
            assert np.all(got_crc[ck] == 99)              # a failed part commits no checksum
            if strict:
                assert np.all(out[by] == 0x5A)            # and, in strict mode, no byte
        else:
            assert np.array_equal(got_crc[ck], want_crc[ck]) and np.array_equal(out[by], a[by])
