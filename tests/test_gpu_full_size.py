"""Parity at the full workload sizes, in the launch configuration the benchmark times.

The engine cache and the incompressible cache are compared with the oracle completely: every
chunk's CRC, every tile table entry and every payload byte of the wire image (the oracle runs the
chunk runs on a thread pool, see oracle_pool.py), the metadata block recomputed with the oracle's
CRC, and the dirty mask against the oracle's byte compare.  The 16 GiB cache is compared on
sampled chunks (the oracle would need minutes for all of it) plus properties that hold at any
size: directory offsets are the running sum of lengths, the decoded shadow equals the cache byte
for byte, a flipped bit is rejected and nothing is installed.
"""
import numpy as np
import pytest
import torch

import oracle
import oracle_pool
from paper_2607_10389_b200 import binding as wm
from paper_2607_10389_b200 import inputs

pytestmark = pytest.mark.gpu

TILE = 16384


class Job:
    """Buffers of one geometry, reused over the calls of a test."""

    def __init__(self, nbytes, chunk):
        self.n, self.chunk = nbytes, chunk
        self.nc = wm.num_chunks(nbytes, chunk)
        self.nt = wm.num_tiles(nbytes)
        self.meta_end = wm.meta_bytes(nbytes, chunk)
        self.cap = wm.wire_bound(nbytes, chunk)
        self.ws = wm.new_workspace(nbytes, chunk)
        self.ws2 = wm.new_workspace(nbytes, chunk)
        self.wire = torch.empty(self.cap, dtype=torch.uint8, device="cuda")
        self.res_e, self.res_d = wm.new_result(), wm.new_result()

    def meta(self):
        m = self.wire[: self.meta_end].cpu().numpy()
        hdr = m[:64]
        directory = m[64: 64 + 16 * self.nc]
        off = directory.view(np.uint64).reshape(self.nc, 2)[:, 0].copy()
        ln = directory.view(np.uint32).reshape(self.nc, 4)[:, 2].copy()
        crc = directory.view(np.uint32).reshape(self.nc, 4)[:, 3].copy()
        tab = m[64 + 16 * self.nc: 64 + 16 * self.nc + 2 * self.nt].view(np.uint16).copy()
        return m, hdr, off, ln, crc, tab


def check_meta_against_oracle(job, m, hdr, off, ln, crc, present):
    """Header, directory sums, metadata CRC and whole-cache CRC, recomputed with the oracle's CRC."""
    assert bytes(hdr[:4]) == b"WMV1"
    assert int(hdr[8:16].view(np.uint64)[0]) == job.n and int(hdr[16:20].view(np.uint32)[0]) == job.chunk
    assert int(hdr[24:28].view(np.uint32)[0]) == job.nc and int(hdr[28:32].view(np.uint32)[0]) == int(present.sum())
    run = np.concatenate([[0], np.cumsum(ln.astype(np.uint64) * present)])[:-1]
    assert np.array_equal(off[present == 1], run[present == 1])
    assert (ln[present == 0] == 0).all()
    payload = int((ln.astype(np.uint64) * present).sum())
    assert int(hdr[32:40].view(np.uint64)[0]) == payload
    assert int(hdr[40:48].view(np.uint64)[0]) == job.meta_end + payload
    z = m.copy()
    z[52:56] = 0
    assert oracle.crc32c(z) == int(hdr[52:56].view(np.uint32)[0])
    acc = int(crc[0])
    for c in range(1, job.nc):
        acc = oracle.crc_combine(acc, int(crc[c]), min(job.chunk, job.n - c * job.chunk))
    assert acc == int(hdr[48:52].view(np.uint32)[0])


def check_chunks_against_oracle(job, cache, chunks, off, ln, crc, tab, entropy=False):
    """Each sampled chunk, encoded alone by the oracle, gives the bytes found in the wire image."""
    tpc = job.chunk // TILE
    for c in chunks:
        lo, hi = c * job.chunk, min((c + 1) * job.chunk, job.n)
        raw = cache[lo:hi].cpu().numpy()
        w1, crc1, r1 = oracle.encode(raw, job.chunk, entropy=entropy)
        assert r1.status == 0
        assert int(crc1[0]) == int(crc[c]) == oracle.crc32c(raw), f"chunk {c}: crc"
        me = oracle.meta_end(hi - lo, job.chunk)
        pay = w1[me: r1.wire_len]
        assert pay.size == int(ln[c]), f"chunk {c}: encoded length"
        a = job.meta_end + int(off[c])
        got = job.wire[a: a + pay.size].cpu().numpy()
        assert np.array_equal(got, pay), f"chunk {c}: payload bytes"
        nt1 = oracle.num_tiles(hi - lo)
        tab1 = w1[64 + 16: 64 + 16 + 2 * nt1].view(np.uint16)
        assert np.array_equal(tab[c * tpc: c * tpc + nt1], tab1), f"chunk {c}: tile table"


def check_whole_image_against_oracle(job, cache, off, ln, crc, tab, present=None, **options):
    """Every present chunk of the image, byte for byte: CRC, encoded length, tile table entries and
    payload against the oracle's encoding of the same bytes; absent chunks have no tiles and no bytes."""
    host = cache.cpu().numpy()
    wire = job.wire.cpu().numpy()
    ocrc, olen, otab, opay = oracle_pool.encode_runs(host, job.chunk, present=present, **options)
    on = np.ones(job.nc, bool) if present is None else np.asarray(present).astype(bool)
    assert np.array_equal(tab, otab), "tile table"
    assert np.array_equal(ln, olen), "encoded lengths"
    assert np.array_equal(crc[on], ocrc[on]), "chunk CRCs"
    bad = [c for c in np.nonzero(on)[0]
           if not np.array_equal(wire[job.meta_end + int(off[c]): job.meta_end + int(off[c]) + int(ln[c])], opay[c])]
    assert not bad, f"payload bytes differ in chunks {bad[:8]} ({len(bad)} in all)"
    return ocrc


def test_engine_cache_full_move_whole_image_against_oracle():
    cfg = inputs.CONFIGS["engine"]
    cur = inputs.make_cache(cfg, "cuda")
    job = Job(cfg.nbytes, cfg.chunk_bytes)
    crc_a = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    crc_b = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    wm.wm_checksum(cur, job.chunk, crc_a, job.ws)
    wm.wm_encode(cur, job.chunk, None, crc_b, job.wire, job.ws, job.res_e)
    r = wm.read_result(job.res_e)
    assert r.ok and r.n_present == job.nc
    assert torch.equal(crc_a, crc_b)
    m, hdr, off, ln, crc, tab = job.meta()
    assert np.array_equal(crc, crc_a.cpu().numpy().view(np.uint32))
    present = np.ones(job.nc, dtype=np.uint64)
    check_meta_against_oracle(job, m, hdr, off, ln, crc, present)
    assert r.wire_len == int(hdr[40:48].view(np.uint64)[0]) and r.cache_crc == int(hdr[48:52].view(np.uint32)[0])
    assert 0.70 < r.wire_len / job.n < 0.80        # the exponent plane carries the saving
    check_whole_image_against_oracle(job, cur, off, ln, crc, tab)

    shadow = torch.zeros(job.n, dtype=torch.uint8, device="cuda")
    crc_dst = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    wm.wm_decode_verify(job.wire, r.wire_len, shadow, job.chunk, crc_dst, job.ws, job.res_d)
    rd = wm.read_result(job.res_d)
    assert rd.ok and rd.cache_crc == r.cache_crc and rd.n_present == job.nc
    assert torch.equal(shadow, cur) and torch.equal(crc_dst, crc_b)


def test_engine_cache_with_entropy_coded_exponents_whole_image_against_oracle():
    """The ENT option at full size: the whole image byte for byte, metadata, round trip, one flipped bit."""
    cfg = inputs.CONFIGS["engine"]
    cur = inputs.make_cache(cfg, "cuda")
    job = Job(cfg.nbytes, cfg.chunk_bytes)
    crc_b = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    wm.entropy_enable(True)
    try:
        wm.wm_encode(cur, job.chunk, None, crc_b, job.wire, job.ws, job.res_e)
        r = wm.read_result(job.res_e)
        assert r.ok and r.n_present == job.nc
        m, hdr, off, ln, crc, tab = job.meta()
        assert int(hdr[6:8].view(np.uint16)[0]) == 4 and ((tab & 0x8000) != 0).mean() > 0.98     # (a few tiles hold a strand the form cannot take)
        present = np.ones(job.nc, dtype=np.uint64)
        check_meta_against_oracle(job, m, hdr, off, ln, crc, present)
        assert 0.68 < r.wire_len / job.n < 0.72        # bit-plane packing: 0.757
        check_whole_image_against_oracle(job, cur, off, ln, crc, tab, entropy=True)
        shadow = torch.zeros(job.n, dtype=torch.uint8, device="cuda")
        crc_dst = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
        wm.wm_decode_verify(job.wire, r.wire_len, shadow, job.chunk, crc_dst, job.ws, job.res_d)
        rd = wm.read_result(job.res_d)
        assert rd.ok and rd.cache_crc == r.cache_crc and torch.equal(shadow, cur) and torch.equal(crc_dst, crc_b)
        # one bit inside a stream of a tile in the middle of the image
        c = job.nc // 2
        at = job.meta_end + int(off[c]) + 9000
        job.wire[at] ^= 0x10
        crc_dst.fill_(7)
        wm.wm_decode_verify(job.wire, r.wire_len, shadow, job.chunk, crc_dst, job.ws, job.res_d)
        rd = wm.read_result(job.res_d)
        assert rd.status_name in ("ERR_CHUNK_CRC", "ERR_DESC") and rd.first_bad_chunk == c and rd.n_bad_chunks == 1
        assert bool((crc_dst == 7).all())
    finally:
        wm.entropy_enable(False)


def test_random_cache_takes_the_raw_path_and_a_flipped_bit_is_rejected():
    cfg = inputs.CONFIGS["random"]
    cur = inputs.make_cache(cfg, "cuda")
    job = Job(cfg.nbytes, cfg.chunk_bytes)
    crc = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    wm.wm_encode(cur, job.chunk, None, crc, job.wire, job.ws, job.res_e)
    r = wm.read_result(job.res_e)
    assert r.ok
    m, hdr, off, ln, dcrc, tab = job.meta()
    # incompressible data: every tile raw, the image is the cache plus its metadata and no more
    assert (tab == 512).all()
    assert r.payload_bytes == job.n and r.wire_len == job.meta_end + job.n
    assert (ln == job.chunk).all()
    check_meta_against_oracle(job, m, hdr, off, ln, dcrc, np.ones(job.nc, dtype=np.uint64))
    check_whole_image_against_oracle(job, cur, off, ln, dcrc, tab)

    shadow = torch.zeros(job.n, dtype=torch.uint8, device="cuda")
    crc_dst = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    wm.wm_decode_verify(job.wire, r.wire_len, shadow, job.chunk, crc_dst, job.ws, job.res_d)
    assert wm.read_result(job.res_d).ok and torch.equal(shadow, cur) and torch.equal(crc_dst, crc)

    # one flipped payload bit: the chunk that holds it is named, and no checksum is installed
    bad_chunk = 611
    pos = job.meta_end + bad_chunk * job.chunk + 123457
    job.wire[pos] ^= 0x10
    crc_dst.fill_(77)
    wm.wm_decode_verify(job.wire, r.wire_len, shadow, job.chunk, crc_dst, job.ws, job.res_d)
    rd = wm.read_result(job.res_d)
    assert rd.status_name == "ERR_CHUNK_CRC" and rd.first_bad_chunk == bad_chunk and rd.n_bad_chunks == 1
    assert (crc_dst == 77).all()
    job.wire[pos] ^= 0x10
    # one flipped metadata bit (a directory length): stopped at the metadata CRC
    job.wire[64 + 16 * 5 + 8] ^= 0x01
    wm.wm_decode_verify(job.wire, r.wire_len, shadow, job.chunk, crc_dst, job.ws, job.res_d)
    assert wm.read_result(job.res_d).status_name == "ERR_META_CRC"
    assert (crc_dst == 77).all()
    job.wire[64 + 16 * 5 + 8] ^= 0x01
    wm.wm_decode_verify(job.wire, r.wire_len, shadow, job.chunk, crc_dst, job.ws, job.res_d)
    assert wm.read_result(job.res_d).ok and torch.equal(crc_dst, crc)


def test_long_context_cache_beyond_4gib_offsets():
    """17 GB cache: payload offsets and tile numbers pass 2^32 bytes / 2^20 tiles."""
    cfg = inputs.CONFIGS["long"]
    free, _ = torch.cuda.mem_get_info()
    if free < 4 * cfg.nbytes:
        pytest.skip("not enough free device memory for the long-context cache")
    cur = inputs.make_cache(cfg, "cuda")
    job = Job(cfg.nbytes, cfg.chunk_bytes)
    crc_a = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    crc_b = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    wm.wm_checksum(cur, job.chunk, crc_a, job.ws)
    wm.wm_encode(cur, job.chunk, None, crc_b, job.wire, job.ws, job.res_e)
    r = wm.read_result(job.res_e)
    assert r.ok and torch.equal(crc_a, crc_b)
    assert r.payload_bytes > (1 << 32)
    m, hdr, off, ln, crc, tab = job.meta()
    check_meta_against_oracle(job, m, hdr, off, ln, crc, np.ones(job.nc, dtype=np.uint64))
    # chunks on both sides of the 4 GiB payload offset, and the ends
    k = int(np.searchsorted(off, 1 << 32))
    check_chunks_against_oracle(job, cur, sorted({0, k - 1, k, k + 1, job.nc - 1}), off, ln, crc, tab)
    shadow = torch.zeros(job.n, dtype=torch.uint8, device="cuda")
    crc_dst = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    wm.wm_decode_verify(job.wire, r.wire_len, shadow, job.chunk, crc_dst, job.ws, job.res_d)
    assert wm.read_result(job.res_d).ok
    assert torch.equal(shadow, cur) and torch.equal(crc_dst, crc_b)


def test_precopy_step_loop_on_two_streams():
    """Twenty generation steps of the engine cache.  Source stream: rewrite three quarters of the
    chunks, diff against the last snapshot, encode only the dirty chunks.  Destination stream:
    decode, verify, install into the destination copy while the source already works on the
    next step.  After every step the destination must equal the source's snapshot."""
    cfg = inputs.CONFIGS["engine"]
    steps = 20
    cur = inputs.make_cache(cfg, "cuda")
    job = Job(cfg.nbytes, cfg.chunk_bytes)
    wires = [job.wire, torch.empty_like(job.wire)]
    src, dstream = torch.cuda.Stream(), torch.cuda.Stream()
    res_d = [wm.new_result(), wm.new_result()]
    crc_src = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    crc_dst = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    dirty = torch.zeros(job.nc, dtype=torch.uint8, device="cuda")
    idx = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    n_dirty = torch.zeros(1, dtype=torch.int32, device="cuda")

    # step 0 of the protocol: a full move brings the destination level with the source
    wm.wm_encode(cur, job.chunk, None, crc_src, wires[0], job.ws, job.res_e)
    r = wm.read_result(job.res_e)
    dst = torch.zeros(job.n, dtype=torch.uint8, device="cuda")
    wm.wm_decode_verify(wires[0], r.wire_len, dst, job.chunk, crc_dst, job.ws, job.res_d)
    assert r.ok and wm.read_result(job.res_d).ok and torch.equal(dst, cur)
    prev = cur.clone()
    torch.cuda.synchronize()

    oracle_steps = {0, 7, 19}
    pending = None                       # (step, result record) of the decode still in flight
    for k in range(steps):
        mask = inputs.step_pattern(job.nc, cfg.shape[0], 0.75, seed=1000 + k)
        wire = wires[(k + 1) % 2]
        with torch.cuda.stream(src):
            inputs.apply_step(cur, job.chunk, mask, seed=5000 + k)
            wm.wm_dirty_diff(cur, prev, job.chunk, dirty, idx, n_dirty, job.ws, stream=src)
            wm.wm_encode(cur, job.chunk, dirty, crc_src, wire, job.ws, job.res_e, stream=src)
            r = wm.read_result(job.res_e)                  # waits for the source stream only
            nd = int(n_dirty.item())
            assert r.ok and r.n_present == nd == int(mask.sum())
            assert torch.equal(dirty.cpu(), mask)
            assert torch.equal(idx[:nd].cpu().long(), torch.nonzero(mask).flatten())
            if k in oracle_steps:
                # the mask and the index list against the oracle's byte compare of the two snapshots,
                # then the whole masked image against the oracle's
                o_dirty, o_idx = oracle_pool.dirty_diff(cur.cpu().numpy(), prev.cpu().numpy(), job.chunk)
                assert np.array_equal(dirty.cpu().numpy(), o_dirty)
                assert np.array_equal(idx[:nd].cpu().numpy().view(np.uint32), o_idx)
                job.wire = wire
                m, hdr, off, ln, crc, tab = job.meta()
                present = mask.numpy().astype(np.uint64)
                check_meta_against_oracle(job, m, hdr, off, ln, crc, present)
                check_whole_image_against_oracle(job, cur, off, ln, crc, tab, present=mask.numpy())
            encoded = torch.cuda.Event()
            encoded.record(src)
        if pending is not None:
            # the previous step's install ran beside this step's source work; settle it now
            dstream.synchronize()
            pk, rec = pending
            rd = wm.read_result(rec)
            assert rd.ok, f"step {pk}: {rd.status_name}"
            assert torch.equal(dst, prev), f"step {pk}: destination differs from the snapshot"
            assert torch.equal(crc_dst, crc_prev)
        with torch.cuda.stream(src):
            prev.copy_(cur, non_blocking=True)             # snapshot for the next diff
            crc_prev = crc_src.clone()
            snap = torch.cuda.Event()
            snap.record(src)
        with torch.cuda.stream(dstream):
            dstream.wait_event(encoded)
            wm.wm_decode_verify(wire, r.wire_len, dst, job.chunk, crc_dst, job.ws2, res_d[k % 2], stream=dstream)
        pending = (k, res_d[k % 2])
        snap.synchronize()
    dstream.synchronize()
    rd = wm.read_result(pending[1])
    assert rd.ok and torch.equal(dst, cur) and torch.equal(crc_dst, crc_src)


def test_engine_cache_as_sixty_leaves_gives_the_flat_image():
    """The engine cache as the model holds it: one key and one value tensor per layer (60 leaves
    of 27.85 MB).  Leaf-mode encode must produce the flat call's image byte for byte, and
    leaf-mode decode must fill separate destination tensors with the source's bytes."""
    cfg = inputs.CONFIGS["engine"]
    cur = inputs.make_cache(cfg, "cuda")
    job = Job(cfg.nbytes, cfg.chunk_bytes)
    n_leaves = cfg.shape[0] * cfg.shape[1]
    leaf_bytes = cfg.nbytes // n_leaves
    assert leaf_bytes % TILE == 0
    leaves = [cur[i * leaf_bytes:(i + 1) * leaf_bytes].clone() for i in range(n_leaves)]
    table = wm.make_leaf_table(leaves)
    crc_flat = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    crc_leaf = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    wm.wm_encode(cur, job.chunk, None, crc_flat, job.wire, job.ws, job.res_e)
    r_flat = wm.read_result(job.res_e)
    wire_leaf = torch.empty_like(job.wire)
    wm.wm_encode_leaves(table, job.n, job.chunk, None, crc_leaf, wire_leaf, job.ws, job.res_e)
    r_leaf = wm.read_result(job.res_e)
    assert r_flat.ok and r_leaf.ok
    assert (r_leaf.wire_len, r_leaf.cache_crc, r_leaf.n_present) == (r_flat.wire_len, r_flat.cache_crc, r_flat.n_present)
    assert torch.equal(wire_leaf[: r_leaf.wire_len], job.wire[: r_flat.wire_len]) and torch.equal(crc_leaf, crc_flat)
    dst = [torch.zeros_like(x) for x in leaves]
    dtable = wm.make_leaf_table(dst)
    crc_dst = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    wm.wm_decode_verify_leaves(wire_leaf, r_leaf.wire_len, dtable, job.n, job.chunk, crc_dst, job.ws, job.res_d)
    assert wm.read_result(job.res_d).ok and torch.equal(crc_dst, crc_flat)
    assert all(torch.equal(a, b) for a, b in zip(dst, leaves))


def test_paper_shaped_leaf_table_gives_the_flat_image_and_scatters_back():
    """450 leaves adding up to 1,670,124,960 bytes: 420 tensors of seeded random sizes with 30
    flags of 2 to 64 bytes between them (the shape of the paper's movable set).  After the first
    flag the tile grid no longer falls on 16-byte boundaries of the leaves, and some tiles cross
    leaves.  The leaf-mode image must be the flat call's byte for byte (which the whole-image test
    ties to the oracle; here chunks around every flag are also compared with the oracle directly),
    and the decode must put every byte back where it came from and touch nothing else."""
    cfg = inputs.CONFIGS["engine"]
    n = inputs.PAPER_CACHE_BYTES
    cur = inputs.make_cache(cfg, "cuda")[:n]
    sizes = inputs.paper_leaf_sizes()
    job = Job(n, cfg.chunk_bytes)
    leaves, o = [], 0
    for k in sizes:
        leaves.append(cur[o:o + k].clone())
        o += k
    table = wm.make_leaf_table(leaves)
    crc_flat = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    crc_leaf = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    wm.wm_encode(cur, job.chunk, None, crc_flat, job.wire, job.ws, job.res_e)
    r_flat = wm.read_result(job.res_e)
    wire_leaf = torch.empty_like(job.wire)
    wm.wm_encode_leaves(table, n, job.chunk, None, crc_leaf, wire_leaf, job.ws, job.res_e)
    r_leaf = wm.read_result(job.res_e)
    assert r_flat.ok and r_leaf.ok
    assert (r_leaf.wire_len, r_leaf.cache_crc, r_leaf.n_present) == (r_flat.wire_len, r_flat.cache_crc, r_flat.n_present)
    assert torch.equal(wire_leaf[: r_leaf.wire_len], job.wire[: r_flat.wire_len]) and torch.equal(crc_leaf, crc_flat)
    # the chunks that hold a flag, and the last (ragged) chunk, against the oracle
    m, hdr, off, ln, crc, tab = job.meta()
    flag_chunks, o = set(), 0
    for k in sizes:
        if k <= 64:
            flag_chunks.add(o // job.chunk)
        o += k
    check_chunks_against_oracle(job, cur, sorted(flag_chunks)[:12] + [job.nc - 1], off, ln, crc, tab)
    # decode into fresh leaves with guard bytes behind each
    store = [torch.full((x.numel() + 16,), 0xC3, dtype=torch.uint8, device="cuda") for x in leaves]
    dst = [b[: x.numel()] for b, x in zip(store, leaves)]
    dtable = wm.make_leaf_table(dst)
    crc_dst = torch.zeros(job.nc, dtype=torch.int32, device="cuda")
    wm.wm_decode_verify_leaves(wire_leaf, r_leaf.wire_len, dtable, n, job.chunk, crc_dst, job.ws, job.res_d)
    assert wm.read_result(job.res_d).ok and torch.equal(crc_dst, crc_flat)
    assert all(torch.equal(a, b) for a, b in zip(dst, leaves))
    assert all(bool((b[-16:] == 0xC3).all()) for b in store), "wrote past the end of a leaf"
