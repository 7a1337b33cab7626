"""Grid independence: tiles are claimed by ticket, so the wire image, the CRC vector and every
result are the same whatever number of thread blocks the main kernels run on.  WM_OPT_BLOCKS caps
that number for callers that share the GPU; here it also serves to prove the independence
(1 encoding block beside the scanner, a handful, half the machine, all of it, more than exist)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_10389_b200 import binding as wm
from paper_2607_10389_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("options,kw", [(0, {}), (wm.OPT_ENTROPY, {"entropy": True}),
                                        (wm.OPT_ZERO_TILES | wm.OPT_ENTROPY, {"entropy": True, "zero_tiles": True})])
def test_same_bytes_at_every_block_count(options, kw):
    cfg = inputs.CONFIGS["engine_small"]
    host = inputs.make_cache(cfg)[: cfg.nbytes - 1234].contiguous()
    host[5 * 65536: 5 * 65536 + 3 * 16384] = 0
    chunk = 65536
    cur = host.cuda()
    n = cur.numel()
    nc = wm.num_chunks(n, chunk)
    rng = np.random.default_rng(11)
    for mask in (None, (rng.random(nc) < 0.75).astype(np.uint8)):
        crc_in = rng.integers(0, 2**32, nc, dtype=np.uint64).astype(np.uint32)
        want_wire, want_crc, want = oracle.encode(host.numpy(), chunk, dirty=mask, crc_in=crc_in, **kw)
        d = None if mask is None else torch.from_numpy(mask).cuda()
        ws, res = wm.new_workspace(n, chunk), wm.new_result()
        wire = torch.zeros(wm.wire_bound(n, chunk), dtype=torch.uint8, device="cuda")
        for blocks in (0, 2, 3, 37, 74, 148, 255):
            crc = torch.from_numpy(crc_in.view(np.int32).copy()).cuda()
            wire.fill_(0xEE)
            wm.wm_encode_opt(cur, chunk, d, crc, wire, ws, res, options | wm.opt_blocks(blocks))
            r = wm.read_result(res)
            assert r.ok and (r.wire_len, r.cache_crc, r.n_present) == (want.wire_len, want.cache_crc, want.n_present), blocks
            assert np.array_equal(wire[: r.wire_len].cpu().numpy(), want_wire), blocks
            assert np.array_equal(crc.cpu().numpy().view(np.uint32), want_crc), blocks
        for blocks in (0, 1, 2, 37, 74, 255):
            dst = host.cuda() if mask is not None else torch.zeros(n, dtype=torch.uint8, device="cuda")
            dst_crc = torch.from_numpy(want_crc.view(np.int32).copy()).cuda() if mask is not None else \
                torch.zeros(nc, dtype=torch.int32, device="cuda")
            wm.wm_decode_verify_opt(wire, r.wire_len, dst, chunk, dst_crc, ws, res,
                                    (options & wm.OPT_ENTROPY) | wm.opt_blocks(blocks))
            rd = wm.read_result(res)
            assert rd.ok and torch.equal(dst, cur), blocks
            assert np.array_equal(dst_crc.cpu().numpy().view(np.uint32), want_crc), blocks


def test_a_block_cap_of_one_is_refused_for_encode():
    cur = torch.zeros(65536, dtype=torch.uint8, device="cuda")
    ws, res = wm.new_workspace(65536, 65536), wm.new_result()
    wire = torch.zeros(wm.wire_bound(65536, 65536), dtype=torch.uint8, device="cuda")
    crc = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(wm.WmError, match="ERR_ARG"):
        wm.wm_encode_opt(cur, 65536, None, crc, wire, ws, res, wm.opt_blocks(1))


def test_placement_is_repeatable_over_many_moves_and_block_counts():
    """Which team gets which tile first changes from run to run and with the number of blocks; the
    bytes must not.  400 moves of a 64 MiB cache, every option set, block counts drawn at random:
    every image equals the first of its option set byte for byte, every round trip returns the
    cache, and no call ends in a timeout."""
    cfg = inputs.CONFIGS["engine_small"]
    g = torch.Generator(device="cuda").manual_seed(77)
    n, chunk = 64 << 20, 1 << 20
    cur = (torch.randn(n // 2, generator=g, device="cuda") * 3).to(torch.bfloat16).view(torch.uint8)
    cur[5 << 20: 6 << 20] = 0
    nc = wm.num_chunks(n, chunk)
    ws, res = wm.new_workspace(n, chunk), wm.new_result()
    wire = torch.zeros(wm.wire_bound(n, chunk), dtype=torch.uint8, device="cuda")
    crc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    dst = torch.zeros(n, dtype=torch.uint8, device="cuda")
    dcrc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    rng = np.random.default_rng(5)
    first = {}
    for i in range(400):
        opt = int(rng.integers(0, 4))
        be, bd = int(rng.choice([0, 2, 5, 37, 74, 111, 148])), int(rng.choice([0, 1, 5, 37, 74, 111, 148]))
        wm.wm_encode_opt(cur, chunk, None, crc, wire, ws, res, opt | wm.opt_blocks(be))
        r = wm.read_result(res)
        assert r.ok, (i, r.status_name)
        img = wire[: r.wire_len]
        if opt not in first:
            first[opt] = (img.clone(), crc.clone())
        assert torch.equal(img, first[opt][0]) and torch.equal(crc, first[opt][1]), (i, opt, be)
        if i % 4 == 0:
            wm.wm_decode_verify_opt(wire, r.wire_len, dst, chunk, dcrc, ws, res, (opt & wm.OPT_ENTROPY) | wm.opt_blocks(bd))
            assert wm.read_result(res).ok and torch.equal(dst, cur) and torch.equal(dcrc, crc), (i, opt, bd)


@pytest.mark.parametrize("chunk_tiles", [1, 3, 4])
@pytest.mark.parametrize("options,kw", [(0, {}), (wm.OPT_ENTROPY | wm.OPT_ZERO_TILES, {"entropy": True, "zero_tiles": True})])
def test_sparse_and_degenerate_masks(chunk_tiles, options, kw):
    """Masked calls claim only the tiles of present chunks.  The masks that stress that: nothing
    present, everything present (with the mask flag), only the short last chunk, everything but
    the last chunk, single chunks, every other chunk; chunk sizes of 1, 3 (no power of two) and
    4 tiles on a cache whose last chunk and last tile are ragged.  Image, CRC vector and result
    are the oracle's; the decode installs exactly the present chunks."""
    TILE = 16384
    chunk = chunk_tiles * TILE
    cfg = inputs.CONFIGS["engine_small"]
    host = inputs.make_cache(cfg)[: 41 * TILE + 777].contiguous()
    host[7 * TILE: 9 * TILE] = 0
    cur = host.cuda()
    n = cur.numel()
    nc = wm.num_chunks(n, chunk)
    masks = {"none": np.zeros(nc, np.uint8), "all": np.ones(nc, np.uint8)}
    m = np.zeros(nc, np.uint8); m[-1] = 1; masks["last only"] = m
    m = np.ones(nc, np.uint8); m[-1] = 0; masks["all but last"] = m
    m = np.zeros(nc, np.uint8); m[0] = 1; masks["first only"] = m
    m = np.zeros(nc, np.uint8); m[nc // 2] = 1; masks["one in the middle"] = m
    masks["every other"] = (np.arange(nc) % 2).astype(np.uint8)
    masks["every other, and the last"] = ((np.arange(nc) % 2 == 0) | (np.arange(nc) == nc - 1)).astype(np.uint8)
    rng = np.random.default_rng(1)
    crc_in = rng.integers(0, 2**32, nc, dtype=np.uint64).astype(np.uint32)
    ws, res = wm.new_workspace(n, chunk), wm.new_result()
    wire = torch.zeros(wm.wire_bound(n, chunk), dtype=torch.uint8, device="cuda")
    old = torch.full((n,), 0x3C, dtype=torch.uint8, device="cuda")
    for name, mask in masks.items():
        want_wire, want_crc, want = oracle.encode(host.numpy(), chunk, dirty=mask, crc_in=crc_in, **kw)
        crc = torch.from_numpy(crc_in.view(np.int32).copy()).cuda()
        wire.fill_(0xEE)
        wm.wm_encode_opt(cur, chunk, torch.from_numpy(mask).cuda(), crc, wire, ws, res, options)
        r = wm.read_result(res)
        assert r.ok and (r.wire_len, r.cache_crc, r.n_present, r.payload_bytes) == \
            (want.wire_len, want.cache_crc, want.n_present, want.payload_bytes), name
        assert np.array_equal(wire[: r.wire_len].cpu().numpy(), want_wire), name
        assert np.array_equal(crc.cpu().numpy().view(np.uint32), want_crc), name
        dst = old.clone()
        dcrc = torch.from_numpy(want_crc.view(np.int32).copy()).cuda()
        wm.wm_decode_verify_opt(wire, r.wire_len, dst, chunk, dcrc, ws, res, options & wm.OPT_ENTROPY)
        assert wm.read_result(res).ok, name
        got = dst.cpu().numpy()
        for c in range(nc):
            lo, hi = c * chunk, min((c + 1) * chunk, n)
            if mask[c]:
                assert np.array_equal(got[lo:hi], host.numpy()[lo:hi]), (name, c)
            else:
                assert (got[lo:hi] == 0x3C).all(), (name, c)
