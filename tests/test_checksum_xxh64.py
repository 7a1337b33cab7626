"""XXH64 as a chunk checksum: the oracle against the `xxhash` package (an independent
implementation) and the catalogue's values; the GPU against the oracle."""
import numpy as np
import pytest

import oracle

xxhash = pytest.importorskip("xxhash")
TILE = 16384


def _bytes(n, seed):
    return np.random.default_rng(seed).integers(0, 256, n, dtype=np.uint8)


def test_oracle_xxh64_known_values_and_library():
    assert oracle.xxh64(b"") == 0xEF46DB3751D8E999                     # the empty string, seed 0
    assert oracle.xxh64(b"123456789") == xxhash.xxh64(b"123456789").intdigest() == 0x8CB841DB40E6AE83
    for n in list(range(0, 70)) + [95, 96, 97, 255, 1000, 4099, 65536, 65536 + 31, 1 << 20]:
        a = _bytes(n, n)
        for seed in (0, 1, 0x9E3779B185EBCA87, 2 ** 64 - 1):
            assert oracle.xxh64(a, seed) == xxhash.xxh64(a.tobytes(), seed=seed).intdigest(), (n, seed)


def test_oracle_chunked_xxh64():
    a = _bytes(5 * TILE + 77, 3)
    got = oracle.checksum_xxh64(a, 2 * TILE, seed=42)
    want = [xxhash.xxh64(a[o:o + 2 * TILE].tobytes(), seed=42).intdigest() for o in range(0, a.size, 2 * TILE)]
    assert got.tolist() == want


SIZES = [1, 3, 4, 7, 8, 9, 31, 32, 33, 63, 64, 95, TILE - 1, TILE, TILE + 1, TILE + 29, 2 * TILE, 3 * TILE + 5536,
         2 * 65536 + 777, 5 * 65536]


@pytest.mark.gpu
@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("chunk", [TILE, 65536])
def test_gpu_xxh64_ragged_sizes(n, chunk):
    import torch
    from paper_2607_10389_b200 import binding as wm
    a = _bytes(n, 5 * n + 3)
    nc = wm.num_chunks(n, chunk)
    for seed in (0, 0xC0FFEE1234567):
        out = torch.full((nc,), 5, dtype=torch.int64, device="cuda")
        wm.wm_checksum_xxh64(torch.from_numpy(a).cuda(), chunk, seed, out)
        assert np.array_equal(out.cpu().numpy().view(np.uint64), oracle.checksum_xxh64(a, chunk, seed))


@pytest.mark.gpu
def test_gpu_xxh64_engine_cache_and_bad_arguments():
    import torch
    from paper_2607_10389_b200 import binding as wm, inputs
    cfg = inputs.CONFIGS["engine"]
    cache = inputs.make_cache(cfg)
    a = cache.numpy().view(np.uint8).reshape(-1)
    nc = wm.num_chunks(cfg.nbytes, cfg.chunk_bytes)
    out = torch.zeros(nc, dtype=torch.int64, device="cuda")
    wm.wm_checksum_xxh64(cache.cuda(), cfg.chunk_bytes, 7, out)
    got = out.cpu().numpy().view(np.uint64)
    for c in (0, 1, nc // 2, nc - 2, nc - 1):                      # the oracle on sampled chunks
        assert int(got[c]) == oracle.xxh64(a[c * cfg.chunk_bytes:(c + 1) * cfg.chunk_bytes], 7)
    lib_all = [xxhash.xxh64(a[o:o + cfg.chunk_bytes].tobytes(), seed=7).intdigest() for o in range(0, a.size, cfg.chunk_bytes)]
    assert got.tolist() == lib_all                                  # and every chunk against the package
    with pytest.raises(wm.WmError, match="ERR_ARG"):
        wm.wm_checksum_xxh64(cache.cuda()[:100], 1000, 0, out)
