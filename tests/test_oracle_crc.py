"""Pins of the oracle's checksum, combination and dirty mask against things that are not the
oracle: published check values, zlib, the CPU's CRC instruction, brute force."""
import ctypes
import os
import subprocess
import zlib

import numpy as np
import pytest

import oracle
from oracle.wm_oracle import POLY_ZLIB

HERE = os.path.dirname(os.path.abspath(__file__))


def _vectors():
    out = []
    for line in open(os.path.join(HERE, "golden", "crc32c_vectors.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        spec, crc = line.split()
        kind, arg = spec.split(":")
        if kind == "ascii":
            data = arg.encode()
        elif kind == "zeros":
            data = bytes(int(arg))
        elif kind == "ones":
            data = b"\xff" * int(arg)
        elif kind == "incr":
            data = bytes(range(int(arg)))
        elif kind == "decr":
            data = bytes(reversed(range(int(arg))))
        else:
            data = b""
        out.append((spec, data, int(crc, 16)))
    return out


@pytest.mark.parametrize("spec,data,want", _vectors())
def test_crc32c_published_vectors(spec, data, want):
    assert oracle.crc_bitwise(data) == want
    assert oracle.crc32c(data) == want


def test_zlib_polynomial_variant():
    rng = np.random.default_rng(7)
    assert oracle.crc_bitwise(b"123456789", POLY_ZLIB) == 0xCBF43926
    for n in (0, 1, 3, 64, 1000, 4097):
        data = rng.integers(0, 256, n, dtype=np.uint8).tobytes()
        assert oracle.crc_bitwise(data, POLY_ZLIB) == zlib.crc32(data)


@pytest.fixture(scope="module")
def hwcrc():
    lib = oracle.hw_crc_library()
    if lib is None:
        pytest.skip("host CPU has no SSE4.2 crc32 instruction")
    return lib


def test_crc32c_against_cpu_instruction(hwcrc):
    rng = np.random.default_rng(11)
    for n in (1, 2, 5, 63, 64, 65, 16384, 65536 + 13, 1 << 20):
        a = rng.integers(0, 256, n, dtype=np.uint8)
        want = hwcrc.hw_crc32c(a.ctypes.data, n)
        assert oracle.crc32c(a) == want == hwcrc.hw_crc32c_u64(a.ctypes.data, n)
        if n <= 70000:
            assert oracle.crc_bitwise(a) == want


def test_combine_is_crc_of_concatenation():
    rng = np.random.default_rng(3)
    for la, lb in ((0, 5), (5, 0), (1, 1), (17, 4096), (65536, 1000), (3, 1 << 20), (100000, 123457)):
        a = rng.integers(0, 256, la, dtype=np.uint8)
        b = rng.integers(0, 256, lb, dtype=np.uint8)
        whole = oracle.crc32c(np.concatenate([a, b]))
        assert oracle.crc_combine(oracle.crc32c(a), oracle.crc32c(b), lb) == whole


def test_combine_matches_zlib_style_identity_on_zero_blocks():
    # crc(A || zeros) obtained two ways
    a = np.arange(100, dtype=np.uint8)
    for nz in (1, 4, 1 << 10, 1 << 16):
        z = np.zeros(nz, dtype=np.uint8)
        assert oracle.crc_combine(oracle.crc32c(a), oracle.crc32c(z), nz) == oracle.crc32c(np.concatenate([a, z]))


def test_chunk_checksums_fold_to_whole_buffer_crc():
    rng = np.random.default_rng(5)
    n, chunk = 5 * 16384 * 4 + 16384 + 777, 4 * 16384
    a = rng.integers(0, 256, n, dtype=np.uint8)
    crcs = oracle.checksum(a, chunk)
    assert len(crcs) == 6
    for c in range(6):
        assert crcs[c] == oracle.crc_bitwise(a[c * chunk:(c + 1) * chunk])
    acc = int(crcs[0])
    for c in range(1, 6):
        acc = oracle.crc_combine(acc, int(crcs[c]), len(a[c * chunk:(c + 1) * chunk]))
    assert acc == oracle.crc32c(a)


def test_chunk_count_of_the_paper_cache():
    # Section 6.3: the movable set is 1,670,124,960 bytes; Appendix G: 399 four-MB chunks
    n = 1_670_124_960
    assert oracle.num_chunks(n, 4 << 20) == 399
    assert n % 16384 == 5536
    assert oracle.num_tiles(n) == n // 16384 + 1


def test_dirty_mask_special_cases():
    rng = np.random.default_rng(9)
    chunk, n = 16384, 16384 * 7 + 100
    a = rng.integers(0, 256, n, dtype=np.uint8)
    d, idx = oracle.dirty_diff(a, a.copy(), chunk)
    assert d.sum() == 0 and len(idx) == 0
    for pos, want in ((0, 0), (chunk - 1, 0), (chunk, 1), (3 * chunk - 1, 2), (n - 1, 7), (7 * chunk, 7)):
        b = a.copy()
        b[pos] ^= 0x10
        d, idx = oracle.dirty_diff(b, a, chunk)
        assert d.tolist() == [1 if c == want else 0 for c in range(8)]
        assert idx.tolist() == [want]
    # rewriting with identical bytes is clean
    b = a.copy()
    b[chunk:2 * chunk] = a[chunk:2 * chunk]
    assert oracle.dirty_diff(b, a, chunk)[0].sum() == 0


def test_dirty_mask_brute_force_and_checksum_variant():
    rng = np.random.default_rng(13)
    chunk, n = 32768, 32768 * 9 + 5000
    a = rng.integers(0, 256, n, dtype=np.uint8)
    b = a.copy()
    touched = [0, 3, 4, 9]
    for c in touched:
        lo = c * chunk
        hi = min(lo + chunk, n)
        b[rng.integers(lo, hi)] ^= 1
    d, idx = oracle.dirty_diff(b, a, chunk)
    brute = [int(not np.array_equal(a[c * chunk:(c + 1) * chunk], b[c * chunk:(c + 1) * chunk])) for c in range(10)]
    assert d.tolist() == brute
    assert idx.tolist() == touched
    # the checksum-vector variant of the mask agrees
    assert ((oracle.checksum(a, chunk) != oracle.checksum(b, chunk)).astype(np.uint8) == d).all()
