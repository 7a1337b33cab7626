"""The oracle is re-entrant: chunk runs pushed through it on a thread pool give exactly what one
single-threaded call over the whole cache gives (the full-size GPU tests rely on this to compare
whole images, not samples)."""
import numpy as np

import oracle
from paper_2607_10389_b200 import inputs

import oracle_pool


def _image_parts(w, nbytes, chunk):
    nc, nt = oracle.num_chunks(nbytes, chunk), oracle.num_tiles(nbytes)
    d = w[64: 64 + 16 * nc]
    off = d.view(np.uint64).reshape(nc, 2)[:, 0]
    ln = d.view(np.uint32).reshape(nc, 4)[:, 2]
    tab = w[64 + 16 * nc: 64 + 16 * nc + 2 * nt].view(np.uint16)
    return off, ln, tab, oracle.meta_end(nbytes, chunk)


def test_pooled_encode_equals_one_call_in_every_option_set():
    cfg = inputs.CONFIGS["engine_small"]
    cache = inputs.make_cache(cfg).numpy()[: cfg.nbytes - 5000]          # ragged last chunk and tile
    cache[3 * (1 << 20): 3 * (1 << 20) + 5 * 16384] = 0                  # a few all-zero tiles
    chunk = 64 * 1024
    nc = oracle.num_chunks(cache.size, chunk)
    rng = np.random.default_rng(5)
    mask = (rng.random(nc) < 0.7).astype(np.uint8)
    for options in ({}, {"entropy": True}, {"zero_tiles": True}, {"entropy": True, "zero_tiles": True}):
        for present in (None, mask):
            w, crc, r = oracle.encode(cache, chunk, dirty=present, **options)
            off, ln, tab, me = _image_parts(w, cache.size, chunk)
            pcrc, plen, ptab, pay = oracle_pool.encode_runs(cache, chunk, present=present, per_run=3, **options)
            assert np.array_equal(plen, ln) and np.array_equal(ptab, tab)
            on = np.ones(nc, bool) if present is None else present.astype(bool)
            assert np.array_equal(pcrc[on], crc[on])
            for c in np.nonzero(on)[0]:
                assert np.array_equal(pay[c], w[me + int(off[c]): me + int(off[c]) + int(ln[c])]), (options, c)
            assert all(pay[c] is None for c in np.nonzero(~on)[0])


def test_pooled_checksum_and_diff_equal_one_call():
    cfg = inputs.CONFIGS["tiny8m"]
    prev = inputs.make_cache(cfg)
    cur, _ = inputs.rewrite_random_chunks(prev, cfg.chunk_bytes, 0.75, seed=3)
    cur, prev = cur.numpy()[:-77], prev.numpy()[:-77]
    assert np.array_equal(oracle_pool.checksum(cur, cfg.chunk_bytes, per_run=5), oracle.checksum(cur, cfg.chunk_bytes))
    d, i = oracle.dirty_diff(cur, prev, cfg.chunk_bytes)
    pd, pi = oracle_pool.dirty_diff(cur, prev, cfg.chunk_bytes, per_run=5)
    assert np.array_equal(pd, d) and np.array_equal(pi, i)
