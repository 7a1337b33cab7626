"""Leaf mode: the cache as a list of tensors.  Its definition is the flat call on the leaves'
concatenation, so the oracle side is that concatenation; the GPU side reads and writes the
leaves in place and must give the same image, checksums, verdicts and bytes."""
import numpy as np
import pytest

import oracle

TILE = 16384


def split_sizes(nbytes, cuts):
    """Leaf sizes for a cache of nbytes cut at the given tile numbers (ascending)."""
    edges = [0] + [c * TILE for c in cuts] + [nbytes]
    return [b - a for a, b in zip(edges[:-1], edges[1:])]


def test_oracle_leaf_calls_are_the_flat_calls_on_the_concatenation():
    rng = np.random.default_rng(7)
    flat = (rng.normal(size=3 * 65536 // 2 + 700).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16).view(np.uint8)
    sizes = split_sizes(flat.size, [1, 5, 6])
    leaves, o = [], 0
    for n in sizes:
        leaves.append(flat[o:o + n].copy())
        o += n
    assert np.array_equal(oracle.flatten_leaves(leaves), flat)
    w0, c0, r0 = oracle.encode(flat, 65536)
    w1, c1, r1 = oracle.encode_leaves(leaves, 65536)
    assert np.array_equal(w0, w1) and np.array_equal(c0, c1) and r0.wire_len == r1.wire_len
    blank = [np.zeros_like(x) for x in leaves]
    out, crc, r = oracle.decode_verify_leaves(w1, blank, 65536)
    assert r.status == 0 and np.array_equal(crc, c0)
    assert all(np.array_equal(a, b) for a, b in zip(out, leaves))
    assert all(not x.any() for x in blank)                     # the caller's arrays are the live state


gpu = pytest.mark.gpu


def _setup(nbytes, chunk, cuts, seed, byte_cuts=False):
    import torch
    from paper_2607_10389_b200 import binding as wm
    g = torch.Generator(device="cuda").manual_seed(seed)
    flat = torch.randn(((nbytes + 1) // 2,), generator=g, device="cuda").to(torch.bfloat16).view(torch.uint8)[:nbytes].contiguous()
    if byte_cuts:
        edges = [0] + list(cuts) + [nbytes]
        sizes = [b - a for a, b in zip(edges[:-1], edges[1:])]
    else:
        sizes = split_sizes(nbytes, cuts)
    assert all(n > 0 for n in sizes) and sum(sizes) == nbytes
    leaves, o = [], 0
    for n in sizes:                      # separate allocations, as an engine's tensors are
        leaves.append(flat[o:o + n].clone())
        o += n
    return torch, wm, flat, leaves


def _flags(start, sizes):
    """Cut positions of a run of small leaves that starts at byte `start`."""
    out, o = [], start
    for n in sizes:
        out.append(o)
        o += n
    out.append(o)
    return out


LEAF_CASES = [
    # leaves that are whole tiles (every tile moves by an aligned bulk copy)
    (5 * 65536 + 3 * TILE + 1000, 65536, [t * TILE for t in (1, 2, 9, 17)]),       # ragged last leaf, chunks straddle leaves
    (40 * TILE, 8 * TILE, [t * TILE for t in (8, 16, 24, 32)]),                    # leaves on chunk boundaries
    (64 * TILE, 65536, [t * TILE for t in range(1, 64)]),                          # one tile per leaf
    (3 * TILE + 2, 65536, []),                                                     # a single leaf
    # leaves of any size: the tile grid falls anywhere inside them
    (23 * TILE + 200, 65536, [3 * TILE + 16, 11 * TILE + 4096 + 32]),              # 16-byte remainders
    (23 * TILE + 200, 65536, [3 * TILE + 8, 11 * TILE + 4096 + 12]),               # 8 and 4-byte remainders
    (23 * TILE + 200, 65536, [3 * TILE + 2, 11 * TILE + 4096 + 6]),                # even remainders
    (23 * TILE + 201, 65536, [3 * TILE + 1, 11 * TILE + 4096 + 7]),                # odd remainders
    # scalar flags between tensors: runs of tiny leaves, a tile that crosses many of them
    (30 * TILE, 4 * TILE, _flags(5 * TILE + 100, [8, 8, 1, 2, 64, 4]) + _flags(17 * TILE - 20, [8] * 6)),
    (12 * TILE + 77, 2 * TILE, _flags(16, [1] * 40) + [7 * TILE - 1, 7 * TILE + 1]),
    (6 * TILE, 65536, list(range(1, 200))),                                        # 199 one-byte leaves, then one large one
    # a last chunk shorter than four bytes, spread over three one-byte leaves
    (2 * 65536 + 3, 65536, [65536 + 5, 2 * 65536, 2 * 65536 + 1, 2 * 65536 + 2]),
    # a leaf whose size is no multiple of 16 and ends exactly on the tile grid (its last tile is walked)
    (9 * TILE, 65536, [8, 5 * TILE]),
]


@gpu
@pytest.mark.parametrize("nbytes,chunk,cuts", LEAF_CASES)
@pytest.mark.parametrize("options", [0, 3])
def test_leaf_encode_and_decode_match_the_oracle(nbytes, chunk, cuts, options):
    torch, wm, flat, leaves = _setup(nbytes, chunk, cuts, seed=nbytes % 1000, byte_cuts=True)
    kw = {"zero_tiles": True, "entropy": True} if options else {}
    nc = wm.num_chunks(nbytes, chunk)
    ws = wm.new_workspace(nbytes, chunk)
    cap = wm.wire_bound(nbytes, chunk)
    res = wm.new_result()
    table = wm.make_leaf_table(leaves)
    for dirty_np in (None, (np.arange(nc) % 3 != 1).astype(np.uint8)):
        crc_in = (np.arange(nc, dtype=np.uint64) * 2654435761 % (1 << 32)).astype(np.uint32)
        want_wire, want_crc, want = oracle.encode(oracle.flatten_leaves([x.cpu().numpy() for x in leaves]), chunk, dirty=dirty_np,
                                                  crc_in=crc_in.astype(np.uint32), **kw)
        wire = torch.full((cap + 64,), 0xA5, dtype=torch.uint8, device="cuda")
        crc = torch.from_numpy(crc_in.astype(np.uint32).view(np.int32).copy()).cuda()
        dirty = None if dirty_np is None else torch.from_numpy(dirty_np).cuda()
        wm.wm_encode_opt(None, chunk, dirty, crc, wire[:cap], ws, res, options, leaf_table=table, nbytes=nbytes)
        r = wm.read_result(res)
        assert (r.status, r.wire_len, r.n_present, r.cache_crc) == (want.status, want.wire_len, want.n_present, want.cache_crc)
        got = wire.cpu().numpy()
        assert np.array_equal(got[: r.wire_len], want_wire) and (got[cap:] == 0xA5).all()
        assert np.array_equal(crc.cpu().numpy().view(np.uint32), want_crc)
        # the flat call gives the same image
        wire2 = torch.zeros(cap, dtype=torch.uint8, device="cuda")
        crc2 = torch.from_numpy(crc_in.astype(np.uint32).view(np.int32).copy()).cuda()
        wm.wm_encode_opt(flat, chunk, dirty, crc2, wire2, ws, res, options)
        assert torch.equal(wire2[: r.wire_len], wire[: r.wire_len])

        # decode into fresh leaves that hold the old content of the absent chunks; canary bytes
        # behind every destination leaf must stay as they are
        old = flat.clone()
        if dirty_np is not None:
            for c in np.nonzero(dirty_np)[0]:
                old[c * chunk: min((c + 1) * chunk, nbytes)] = 0x11
        dst_store, dst_leaves, o = [], [], 0
        for x in leaves:
            buf = torch.full((x.numel() + 32,), 0xC3, dtype=torch.uint8, device="cuda")
            buf[: x.numel()] = old[o:o + x.numel()]
            dst_store.append(buf)
            dst_leaves.append(buf[: x.numel()])
            o += x.numel()
        dtable = wm.make_leaf_table(dst_leaves)
        for strict in (0, wm.OPT_STRICT):
            dcrc = crc.clone()
            wm.wm_decode_verify_opt(wire, r.wire_len, None, chunk, dcrc, ws, res, (options & 2) | strict, leaf_table=dtable, nbytes=nbytes)
            rd = wm.read_result(res)
            assert rd.ok and rd.cache_crc == want.cache_crc
            assert all(torch.equal(a, b) for a, b in zip(dst_leaves, leaves))
            assert all(bool((b[-32:] == 0xC3).all()) for b in dst_store), "wrote past the end of a leaf"
        # one flipped payload bit on the way into the leaves: the oracle's verdict on the same image
        wire[r.wire_len - 5] ^= 4
        wm.wm_decode_verify_opt(wire, r.wire_len, None, chunk, dcrc, ws, res, options & 2, leaf_table=dtable, nbytes=nbytes)
        _, _, o_res = oracle.decode_verify(wire[: r.wire_len].cpu().numpy(), nbytes, chunk, dst=old.cpu().numpy(),
                                           dst_crc=crc.cpu().numpy().view(np.uint32), expect_entropy=bool(options & 2))
        rd = wm.read_result(res)
        assert (rd.status, rd.first_bad_chunk, rd.n_bad_chunks) == (o_res.status, o_res.first_bad_chunk, o_res.n_bad_chunks)


@gpu
def test_leaf_table_that_breaks_the_rules_is_rejected():
    torch, wm, flat, leaves = _setup(8 * TILE, 65536, [2, 5], seed=3)
    nbytes, chunk = 8 * TILE, 65536
    nc = wm.num_chunks(nbytes, chunk)
    ws, res = wm.new_workspace(nbytes, chunk), wm.new_result()
    cap = wm.wire_bound(nbytes, chunk)
    wire = torch.zeros(cap, dtype=torch.uint8, device="cuda")
    crc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    good = wm.make_leaf_table(leaves)
    wm.wm_encode_leaves(good, nbytes, chunk, None, crc, wire, ws, res)
    r = wm.read_result(res)
    assert r.ok
    bad_tables = []
    t = good.clone(); t[2, 1] += TILE; bad_tables.append(t)                        # sizes do not add up
    t = good.clone(); t[1, 0] += 4; bad_tables.append(t)                           # misaligned leaf
    t = good.clone(); t[1, 1] = 0; bad_tables.append(t)                            # empty leaf
    t = good.clone(); t[1, 0] = 0; bad_tables.append(t)                            # null leaf
    # two sizes that wrap around 2^64 to the right total: -16384 and what is left + 16384
    t = good.clone(); t[0, 1] = -TILE; t[1, 1] = int(good[0, 1]) + int(good[1, 1]) + TILE; bad_tables.append(t)
    for t in bad_tables:
        wm.wm_encode_leaves(t, nbytes, chunk, None, crc, wire, ws, res)
        assert wm.read_result(res).status_name == "ERR_ARG"
        assert wm.workspace_status(ws) == -1
    # decode: a bad destination table is refused before anything is written
    wm.wm_encode_leaves(good, nbytes, chunk, None, crc, wire, ws, res)
    dst = [torch.full_like(x, 0x33) for x in leaves]
    for t in bad_tables:
        dt = wm.make_leaf_table(dst)
        dt[:, 1] = t[:, 1]
        if not torch.equal(t[:, 0], good[:, 0]):
            dt[1, 0] = 0 if int(t[1, 0]) == 0 else dt[1, 0] + 4
        dcrc = torch.zeros(nc, dtype=torch.int32, device="cuda")
        wm.wm_decode_verify_leaves(wire, r.wire_len, dt, nbytes, chunk, dcrc, ws, res)
        assert wm.read_result(res).status_name == "ERR_ARG"
        assert all((x == 0x33).all() for x in dst) and not dcrc.any()


@gpu
def test_a_table_that_cuts_more_tiles_than_the_side_buffer_holds_is_refused():
    """Tiles that cross leaf boundaries go through a side buffer of 2048 slots; 3000 leaves of one
    tile and 16 bytes each cut 2999 tiles, which is refused as an argument error (the same cache as
    1500 leaves of twice that size is accepted)."""
    import torch
    from paper_2607_10389_b200 import binding as wm
    k = 3000
    leaf = TILE + 16
    nbytes, chunk = k * leaf, 4 * TILE
    flat = torch.randint(0, 256, (nbytes,), dtype=torch.uint8, device="cuda")
    nc = wm.num_chunks(nbytes, chunk)
    ws, res = wm.new_workspace(nbytes, chunk), wm.new_result()
    wire = torch.zeros(wm.wire_bound(nbytes, chunk), dtype=torch.uint8, device="cuda")
    crc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    many = wm.make_leaf_table([flat[i * leaf:(i + 1) * leaf] for i in range(k)])
    wm.wm_encode_leaves(many, nbytes, chunk, None, crc, wire, ws, res)
    assert wm.read_result(res).status_name == "ERR_ARG"
    fewer = wm.make_leaf_table([flat[i * 2 * leaf:(i + 1) * 2 * leaf] for i in range(k // 2)])
    wm.wm_encode_leaves(fewer, nbytes, chunk, None, crc, wire, ws, res)
    r = wm.read_result(res)
    wire2 = torch.zeros_like(wire)
    wm.wm_encode(flat, chunk, None, crc, wire2, ws, res)
    assert r.ok and torch.equal(wire[: r.wire_len], wire2[: r.wire_len])
    dst = torch.zeros_like(flat)
    dmany = wm.make_leaf_table([dst[i * leaf:(i + 1) * leaf] for i in range(k)])
    dcrc = torch.zeros_like(crc)
    wm.wm_decode_verify_leaves(wire, r.wire_len, dmany, nbytes, chunk, dcrc, ws, res)
    assert wm.read_result(res).status_name == "ERR_ARG" and not bool(dst.any()) and not bool(dcrc.any())


def test_append_only_workload_dirties_only_the_chunks_that_hold_the_new_tokens():
    from paper_2607_10389_b200 import inputs
    cfg = inputs.CONFIGS["llm_append_small"]
    a = inputs.make_cache(cfg, "cpu")
    prev, mask = inputs.before_append(a, cfg, 16)
    d, idx = oracle.dirty_diff(a.numpy(), prev.numpy(), cfg.chunk_bytes)
    assert np.array_equal(d, mask.numpy()) and 0 < int(d.sum()) <= d.size // 8
    plain = oracle.encode(a.numpy(), cfg.chunk_bytes)[2]
    opt = oracle.encode(a.numpy(), cfg.chunk_bytes, zero_tiles=True)[2]
    # three quarters of the window are unused: without the option they still cost half their size
    assert 0.5 < plain.wire_len / cfg.nbytes < 0.6 and 0.15 < opt.wire_len / cfg.nbytes < 0.25


@gpu
def test_append_only_step_with_zero_tiles_matches_the_oracle():
    import torch
    from paper_2607_10389_b200 import binding as wm
    from paper_2607_10389_b200 import inputs
    cfg = inputs.CONFIGS["llm_append_small"]
    cur = inputs.make_cache(cfg, "cuda")
    prev, mask = inputs.before_append(cur, cfg, 16)
    n, chunk = cfg.nbytes, cfg.chunk_bytes
    nc = wm.num_chunks(n, chunk)
    ws, res = wm.new_workspace(n, chunk), wm.new_result()
    cap = wm.wire_bound(n, chunk)
    dirty = torch.zeros(nc, dtype=torch.uint8, device="cuda")
    nd = torch.zeros(1, dtype=torch.int32, device="cuda")
    wm.wm_dirty_diff(cur, prev, chunk, dirty, None, nd, ws)
    assert torch.equal(dirty.cpu(), mask)
    crc_prev = torch.from_numpy(oracle.checksum(prev.cpu().numpy(), chunk).view(np.int32).copy()).cuda()
    wm.zero_tiles_enable(True)
    try:
        for d_np, d_dev, crc0 in ((None, None, torch.zeros_like(crc_prev)), (mask.numpy(), dirty, crc_prev)):
            want_wire, want_crc, want = oracle.encode(cur.cpu().numpy(), chunk, dirty=d_np,
                                                      crc_in=crc0.cpu().numpy().view(np.uint32), zero_tiles=True)
            wire = torch.zeros(cap, dtype=torch.uint8, device="cuda")
            crc = crc0.clone()
            wm.wm_encode(cur, chunk, d_dev, crc, wire, ws, res)
            r = wm.read_result(res)
            assert (r.status, r.wire_len, r.n_present, r.cache_crc) == (want.status, want.wire_len, want.n_present, want.cache_crc)
            assert np.array_equal(wire[: r.wire_len].cpu().numpy(), want_wire)
            assert np.array_equal(crc.cpu().numpy().view(np.uint32), want_crc)
            dst = prev.clone() if d_np is not None else torch.full_like(cur, 0x77)
            dcrc = crc_prev.clone()
            wm.wm_decode_verify(wire, r.wire_len, dst, chunk, dcrc, ws, res)
            assert wm.read_result(res).ok and torch.equal(dst, cur)
    finally:
        wm.zero_tiles_enable(False)


def test_append_only_schedule_fills_the_window_and_has_an_all_clean_step():
    """The window fills from 0.249 to 0.727 over a run of appends (Section 3.3); every step dirties
    exactly the chunks that hold its new tokens, the step that appends nothing is all clean and its
    image is metadata only."""
    from paper_2607_10389_b200 import inputs
    cfg = inputs.CONFIGS["llm_append_small"]
    cur = inputs.make_cache(cfg, "cpu")
    sched = inputs.append_schedule(cfg, 6)
    assert sched[0][0] == inputs.filled_tokens(cfg) and sum(c for _, c in sched) == round(0.727 * cfg.shape[3]) - sched[0][0]
    assert [c for _, c in sched].count(0) == 1
    crc = oracle.checksum(cur.numpy(), cfg.chunk_bytes)
    for k, (first, count) in enumerate(sched):
        prev = cur.clone()
        mask = inputs.append_tokens(cur, cfg, first, count, seed=40 + k)
        d, _ = oracle.dirty_diff(cur.numpy(), prev.numpy(), cfg.chunk_bytes)
        assert np.array_equal(d, mask.numpy())
        wire, crc, res = oracle.encode(cur.numpy(), cfg.chunk_bytes, dirty=d, crc_in=crc, zero_tiles=True)
        if count == 0:
            assert res.n_present == 0 and res.payload_bytes == 0 and res.wire_len == oracle.meta_end(cfg.nbytes, cfg.chunk_bytes)
        else:
            assert 0 < res.n_present <= d.size // 2
        out, _, r = oracle.decode_verify(wire, cfg.nbytes, cfg.chunk_bytes, dst=prev.numpy(), dst_crc=oracle.checksum(prev.numpy(), cfg.chunk_bytes))
        assert r.status == 0 and np.array_equal(out, cur.numpy())


@gpu
def test_append_only_schedule_on_the_gpu_matches_the_oracle_step_by_step():
    import torch
    from paper_2607_10389_b200 import binding as wm
    from paper_2607_10389_b200 import inputs
    cfg = inputs.CONFIGS["llm_append_small"]
    cur = inputs.make_cache(cfg, "cuda")
    n, chunk = cfg.nbytes, cfg.chunk_bytes
    nc = wm.num_chunks(n, chunk)
    ws, res = wm.new_workspace(n, chunk), wm.new_result()
    wire = torch.zeros(wm.wire_bound(n, chunk), dtype=torch.uint8, device="cuda")
    dirty = torch.zeros(nc, dtype=torch.uint8, device="cuda")
    nd = torch.zeros(1, dtype=torch.int32, device="cuda")
    crc = torch.from_numpy(oracle.checksum(cur.cpu().numpy(), chunk).view(np.int32).copy()).cuda()
    dst, dcrc = cur.clone(), crc.clone()
    for k, (first, count) in enumerate(inputs.append_schedule(cfg, 6)):
        prev = cur.clone()
        mask = inputs.append_tokens(cur, cfg, first, count, seed=40 + k)
        wm.wm_dirty_diff(cur, prev, chunk, dirty, None, nd, ws)
        assert torch.equal(dirty.cpu(), mask) and int(nd.item()) == int(mask.sum())
        want_wire, want_crc, want = oracle.encode(cur.cpu().numpy(), chunk, dirty=mask.numpy(),
                                                  crc_in=crc.cpu().numpy().view(np.uint32), zero_tiles=True)
        wm.wm_encode_opt(cur, chunk, dirty, crc, wire, ws, res, wm.OPT_ZERO_TILES)
        r = wm.read_result(res)
        assert (r.status, r.wire_len, r.n_present, r.cache_crc) == (want.status, want.wire_len, want.n_present, want.cache_crc)
        assert np.array_equal(wire[: r.wire_len].cpu().numpy(), want_wire)
        assert np.array_equal(crc.cpu().numpy().view(np.uint32), want_crc)
        if count == 0:
            assert r.payload_bytes == 0
        wm.wm_decode_verify_opt(wire, r.wire_len, dst, chunk, dcrc, ws, res, 0)
        assert wm.read_result(res).ok and torch.equal(dst, cur) and torch.equal(dcrc, crc)
