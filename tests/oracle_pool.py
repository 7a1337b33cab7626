"""The oracle over a whole multi-gigabyte cache, in seconds: chunks are independent in every step
of the path, so the cache is cut into runs of whole chunks and each run goes through the
oracle's ordinary single-threaded functions on a thread pool (ctypes releases the interpreter
lock during the calls; the C functions keep no state between calls).  Nothing here computes
anything itself: it slices, calls ``oracle.*`` and concatenates.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

import oracle

TILE = 16384


def _runs(n_chunks: int, per_run: int):
    return [(c0, min(c0 + per_run, n_chunks)) for c0 in range(0, n_chunks, per_run)]


def _pool():
    return ThreadPoolExecutor(max_workers=max(1, os.cpu_count() or 1))


def checksum(cache: np.ndarray, chunk_bytes: int, per_run: int = 8) -> np.ndarray:
    nc = oracle.num_chunks(cache.size, chunk_bytes)
    with _pool() as ex:
        parts = ex.map(lambda r: oracle.checksum(cache[r[0] * chunk_bytes: r[1] * chunk_bytes], chunk_bytes), _runs(nc, per_run))
        return np.concatenate(list(parts))


def dirty_diff(cache: np.ndarray, prev: np.ndarray, chunk_bytes: int, per_run: int = 8):
    """(dirty u8[n_chunks], ascending indices of the dirty chunks)."""
    nc = oracle.num_chunks(cache.size, chunk_bytes)
    with _pool() as ex:
        parts = ex.map(lambda r: oracle.dirty_diff(cache[r[0] * chunk_bytes: r[1] * chunk_bytes],
                                                   prev[r[0] * chunk_bytes: r[1] * chunk_bytes], chunk_bytes)[0], _runs(nc, per_run))
        dirty = np.concatenate(list(parts))
    return dirty, np.nonzero(dirty)[0].astype(np.uint32)


def encode_runs(cache: np.ndarray, chunk_bytes: int, present=None, per_run: int = 8, **options):
    """Every present chunk encoded by the oracle.  Returns per chunk: crc u32[n_chunks] (0 for absent
    chunks), enc_len u32[n_chunks], the tile table u16[n_tiles] and a list `payload[c]` of the
    chunk's encoded bytes (None for absent chunks).  A run is encoded as a cache of its own with
    the same chunk size, which gives the same per-chunk bytes as the whole cache would."""
    n = cache.size
    nc = oracle.num_chunks(n, chunk_bytes)
    tpc = chunk_bytes // TILE
    present = np.ones(nc, dtype=np.uint8) if present is None else np.asarray(present, dtype=np.uint8)

    def one(run):
        c0, c1 = run
        lo, hi = c0 * chunk_bytes, min(c1 * chunk_bytes, n)
        sub = cache[lo:hi]
        mask = present[c0:c1]
        if not mask.any():
            return run, None
        w, crc, r = oracle.encode(sub, chunk_bytes, dirty=None if mask.all() else mask, **options)
        assert r.status == 0
        k = c1 - c0
        directory = w[64: 64 + 16 * k]
        off = directory.view(np.uint64).reshape(k, 2)[:, 0]
        ln = directory.view(np.uint32).reshape(k, 4)[:, 2]
        nt = oracle.num_tiles(hi - lo)
        tab = w[64 + 16 * k: 64 + 16 * k + 2 * nt].view(np.uint16).copy()
        me = oracle.meta_end(hi - lo, chunk_bytes)
        pay = [w[me + int(off[i]): me + int(off[i]) + int(ln[i])].copy() if mask[i] else None for i in range(k)]
        return run, (crc * mask, ln.copy(), tab, pay)

    crc_all = np.zeros(nc, dtype=np.uint32)
    len_all = np.zeros(nc, dtype=np.uint32)
    tab_all = np.zeros(oracle.num_tiles(n), dtype=np.uint16)
    payload = [None] * nc
    with _pool() as ex:
        for (c0, c1), out in ex.map(one, _runs(nc, per_run)):
            if out is None:
                continue
            crc, ln, tab, pay = out
            crc_all[c0:c1] = crc
            len_all[c0:c1] = ln
            tab_all[c0 * tpc: c0 * tpc + tab.size] = tab
            payload[c0:c1] = pay
    return crc_all, len_all, tab_all, payload
