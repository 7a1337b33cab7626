"""wm_checksum_poly: the checksum step with the CRC-32 of zlib as the second polynomial.

The oracle's definition is the bit-at-a-time CRC per chunk; `zlib.crc32` (a library that shares
nothing with it) pins that definition, and the GPU must agree with both, bit for bit.
"""
import zlib

import numpy as np
import pytest

import oracle
from oracle.wm_oracle import POLY_CRC32C, POLY_ZLIB

TILE = 16384


def _bytes(n, seed):
    return np.random.default_rng(seed).integers(0, 256, n, dtype=np.uint8)


def _zlib_chunks(a, chunk):
    return np.array([zlib.crc32(a[o: o + chunk].tobytes()) for o in range(0, a.size, chunk)], dtype=np.uint32)


@pytest.mark.parametrize("n,chunk", [(1, TILE), (TILE + 3, TILE), (3 * 65536 + 777, 65536), (5 * TILE, 2 * TILE)])
def test_oracle_poly_checksum_is_zlib_and_crc32c(n, chunk):
    a = _bytes(n, n)
    assert np.array_equal(oracle.checksum_poly(a, chunk, POLY_ZLIB), _zlib_chunks(a, chunk))
    assert np.array_equal(oracle.checksum_poly(a, chunk, POLY_CRC32C), oracle.checksum(a, chunk))
    # the check value of the CRC-32 catalogue entry for this polynomial
    assert oracle.checksum_poly(np.frombuffer(b"123456789", dtype=np.uint8), TILE, POLY_ZLIB)[0] == 0xCBF43926


SIZES = [1, 2, 3, 4, 5, 15, 16, 17, 4095, TILE - 1, TILE, TILE + 1, TILE + 3, 2 * TILE, 3 * TILE + 5536,
         2 * 65536 + 777, 5 * 65536]


@pytest.mark.gpu
@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("chunk", [TILE, 65536])
def test_gpu_zlib_checksum_ragged_sizes(n, chunk):
    import torch
    from paper_2607_10389_b200 import binding as wm
    a = _bytes(n, 7 * n + 1)
    dev = torch.from_numpy(a).cuda()
    nc = wm.num_chunks(n, chunk)
    ws = wm.new_workspace(n, chunk)
    for poly, want in ((wm.POLY_ZLIB, oracle.checksum_poly(a, chunk, POLY_ZLIB)),
                       (wm.POLY_CRC32C, oracle.checksum(a, chunk))):
        out = torch.full((nc,), 5, dtype=torch.int32, device="cuda")
        wm.wm_checksum_poly(dev, chunk, poly, out, ws)
        assert np.array_equal(out.cpu().numpy().view(np.uint32), want)
    assert np.array_equal(oracle.checksum_poly(a, chunk, POLY_ZLIB), _zlib_chunks(a, chunk))


@pytest.mark.gpu
def test_gpu_zlib_checksum_unknown_polynomial_is_refused():
    import torch
    from paper_2607_10389_b200 import binding as wm
    dev = torch.zeros(4 * TILE, dtype=torch.uint8, device="cuda")
    out = torch.full((4,), 5, dtype=torch.int32, device="cuda")
    ws = wm.new_workspace(4 * TILE, TILE)
    with pytest.raises(wm.WmError, match="ERR_ARG"):
        wm.wm_checksum_poly(dev, TILE, 2, out, ws)
    torch.cuda.synchronize()
    assert bool((out == 5).all())


@pytest.mark.gpu
def test_gpu_zlib_checksum_engine_cache():
    """Full size, the launch configuration the benchmark times: every chunk against zlib, a sample
    of chunks (first, a middle one, the ragged last) against the oracle's bitwise definition."""
    import torch
    from paper_2607_10389_b200 import binding as wm, inputs
    cfg = inputs.CONFIGS["engine"]
    cache = inputs.make_cache(cfg)
    a = cache.numpy().view(np.uint8).reshape(-1)
    n, chunk = cfg.nbytes, cfg.chunk_bytes
    nc = wm.num_chunks(n, chunk)
    out = torch.zeros(nc, dtype=torch.int32, device="cuda")
    wm.wm_checksum_poly(cache.cuda(), chunk, wm.POLY_ZLIB, out, wm.new_workspace(n, chunk))
    got = out.cpu().numpy().view(np.uint32)
    assert np.array_equal(got, _zlib_chunks(a, chunk))
    for c in (0, nc // 2, nc - 1):
        assert got[c] == oracle.crc_bitwise(a[c * chunk: (c + 1) * chunk], POLY_ZLIB)
