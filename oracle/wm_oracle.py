"""ctypes front end of ``wm_oracle.c`` (test infrastructure only; see the C file's header).

Every function takes and returns numpy arrays on the host.  The shared object is built on
first use into ``oracle/_build/`` with gcc; ``build()`` may be called ahead of time.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wm_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_SO = os.path.join(_OUT_DIR, "libwm_oracle.so")
_lib = None

POLY_CRC32C = 0x82F63B78
POLY_ZLIB = 0xEDB88320

STATUS = {
    0: "OK", -1: "ERR_ARG", -2: "ERR_CAPACITY", -3: "ERR_FORMAT", -4: "ERR_META_CRC",
    -5: "ERR_STRUCT", -6: "ERR_DESC", -7: "ERR_CHUNK_CRC", -8: "ERR_STALE", -9: "ERR_CACHE_CRC",
}


class _CResult(ctypes.Structure):
    _fields_ = [
        ("status", ctypes.c_int32), ("first_bad_chunk", ctypes.c_uint32),
        ("n_bad_chunks", ctypes.c_uint32), ("n_present", ctypes.c_uint32),
        ("wire_len", ctypes.c_uint64), ("payload_bytes", ctypes.c_uint64),
        ("cache_crc", ctypes.c_uint32), ("reserved", ctypes.c_uint32),
    ]


@dataclass
class Result:
    status: int
    first_bad_chunk: int
    n_bad_chunks: int
    n_present: int
    wire_len: int
    payload_bytes: int
    cache_crc: int

    @property
    def status_name(self) -> str:
        return STATUS.get(self.status, str(self.status))


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, no intrinsics) and return the path of the library."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        os.makedirs(_OUT_DIR, exist_ok=True)
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    u8p, u32p = ctypes.c_void_p, ctypes.c_void_p
    u64, u32 = ctypes.c_uint64, ctypes.c_uint32
    lib.wmo_crc_bitwise.restype = u32
    lib.wmo_crc_bitwise.argtypes = [u8p, u64, u32]
    lib.wmo_crc32c.restype = u32
    lib.wmo_crc32c.argtypes = [u8p, u64]
    lib.wmo_crc_combine.restype = u32
    lib.wmo_crc_combine.argtypes = [u32, u32, u64]
    for name in ("wmo_num_chunks", "wmo_meta_end", "wmo_wire_bound"):
        getattr(lib, name).restype = u64
        getattr(lib, name).argtypes = [u64, u32]
    lib.wmo_num_tiles.restype = u64
    lib.wmo_num_tiles.argtypes = [u64]
    lib.wmo_xxh64.restype = ctypes.c_uint64
    lib.wmo_xxh64.argtypes = [u8p, u64, u64]
    lib.wmo_checksum_xxh64.restype = ctypes.c_int
    lib.wmo_checksum_xxh64.argtypes = [u8p, u64, u32, u64, ctypes.c_void_p]
    lib.wmo_checksum.restype = ctypes.c_int
    lib.wmo_checksum.argtypes = [u8p, u64, u32, u32p]
    lib.wmo_dirty_diff.restype = ctypes.c_int
    lib.wmo_dirty_diff.argtypes = [u8p, u8p, u64, u32, u8p, u32p, u32p]
    lib.wmo_encode.restype = ctypes.c_int
    lib.wmo_encode.argtypes = [u8p, u64, u32, u8p, u32p, u8p, u64, ctypes.POINTER(_CResult)]
    lib.wmo_encode_opt.restype = ctypes.c_int
    lib.wmo_encode_opt.argtypes = [u8p, u64, u32, u8p, u32p, u8p, u64, ctypes.c_int, ctypes.POINTER(_CResult)]
    lib.wmo_decode_verify.restype = ctypes.c_int
    lib.wmo_decode_verify.argtypes = [u8p, u64, u8p, u64, u32, u32p, ctypes.POINTER(_CResult)]
    lib.wmo_decode_verify_opt.restype = ctypes.c_int
    lib.wmo_decode_verify_opt.argtypes = [u8p, u64, u8p, u64, u32, u32p, ctypes.c_int, ctypes.POINTER(_CResult)]
    _lib = lib
    return lib


def _bytes_view(a) -> np.ndarray:
    if isinstance(a, (bytes, bytearray, memoryview)):
        return np.frombuffer(bytes(a), dtype=np.uint8)
    a = np.ascontiguousarray(a)
    return a.view(np.uint8).reshape(-1)


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def _result(r: _CResult) -> Result:
    return Result(r.status, r.first_bad_chunk, r.n_bad_chunks, r.n_present, r.wire_len,
                  r.payload_bytes, r.cache_crc)


_hw = None


def hw_crc_library():
    """The SSE4.2 `crc32` instruction behind two C functions (hw_crc32c: a byte per instruction,
    hw_crc32c_u64: eight), compiled on first use; None where the host CPU lacks the instruction.
    A second opinion for the pins and a strong CPU baseline; the oracle itself never uses it."""
    global _hw
    if _hw is None:
        try:
            has = "sse4_2" in open("/proc/cpuinfo").read()
        except OSError:
            has = False
        if not has:
            _hw = False
        else:
            os.makedirs(_OUT_DIR, exist_ok=True)
            so = os.path.join(_OUT_DIR, "libhwcrc.so")
            src = os.path.join(os.path.dirname(_SRC), "hwcrc.c")
            if not os.path.exists(so) or os.path.getmtime(so) < os.path.getmtime(src):
                tmp = so + f".{os.getpid()}.tmp"
                subprocess.check_call(["gcc", "-O2", "-msse4.2", "-shared", "-fPIC", "-o", tmp, src])
                os.replace(tmp, so)
            lib = ctypes.CDLL(so)
            for name in ("hw_crc32c", "hw_crc32c_u64"):
                getattr(lib, name).restype = ctypes.c_uint32
                getattr(lib, name).argtypes = [ctypes.c_void_p, ctypes.c_uint64]
            _hw = lib
    return _hw or None


def crc_bitwise(data, poly: int = POLY_CRC32C) -> int:
    b = _bytes_view(np.frombuffer(data, dtype=np.uint8) if isinstance(data, (bytes, bytearray)) else data)
    return int(_load().wmo_crc_bitwise(_ptr(b), b.size, poly))


def crc32c(data) -> int:
    b = _bytes_view(np.frombuffer(data, dtype=np.uint8) if isinstance(data, (bytes, bytearray)) else data)
    return int(_load().wmo_crc32c(_ptr(b), b.size))


def crc_combine(crc_a: int, crc_b: int, len_b: int) -> int:
    return int(_load().wmo_crc_combine(crc_a, crc_b, len_b))


def num_chunks(nbytes: int, chunk_bytes: int) -> int:
    return int(_load().wmo_num_chunks(nbytes, chunk_bytes))


def num_tiles(nbytes: int) -> int:
    return int(_load().wmo_num_tiles(nbytes))


def meta_end(nbytes: int, chunk_bytes: int) -> int:
    return int(_load().wmo_meta_end(nbytes, chunk_bytes))


def wire_bound(nbytes: int, chunk_bytes: int) -> int:
    return int(_load().wmo_wire_bound(nbytes, chunk_bytes))


def _check(status: int, what: str) -> None:
    if status == -1:
        raise ValueError(f"oracle {what}: bad argument")


def checksum(cache, chunk_bytes: int) -> np.ndarray:
    b = _bytes_view(cache)
    out = np.zeros(num_chunks(b.size, chunk_bytes), dtype=np.uint32)
    _check(_load().wmo_checksum(_ptr(b), b.size, chunk_bytes, _ptr(out)), "checksum")
    return out


def xxh64(data, seed: int = 0) -> int:
    """XXH64 of a byte string (the published algorithm, written out in the C file)."""
    b = _bytes_view(data)
    return int(_load().wmo_xxh64(_ptr(b), b.size, seed & 0xFFFFFFFFFFFFFFFF))


def checksum_xxh64(cache, chunk_bytes: int, seed: int = 0) -> np.ndarray:
    """XXH64 of every chunk (u64[n_chunks])."""
    b = _bytes_view(cache)
    out = np.zeros(num_chunks(b.size, chunk_bytes), dtype=np.uint64)
    _check(_load().wmo_checksum_xxh64(_ptr(b), b.size, chunk_bytes, seed & 0xFFFFFFFFFFFFFFFF, out.ctypes.data), "checksum_xxh64")
    return out


def checksum_poly(cache, chunk_bytes: int, poly: int) -> np.ndarray:
    """The checksum step with another polynomial: the bit-at-a-time definition, chunk by chunk."""
    b = _bytes_view(cache)
    n = num_chunks(b.size, chunk_bytes)
    return np.array([crc_bitwise(b[c * chunk_bytes: (c + 1) * chunk_bytes], poly) for c in range(n)], dtype=np.uint32)


def dirty_diff(cache, prev, chunk_bytes: int):
    """Return (dirty u8[n_chunks], dirty_idx u32[n_dirty])."""
    a, p = _bytes_view(cache), _bytes_view(prev)
    if a.size != p.size:
        raise ValueError("snapshots differ in size")
    nc = num_chunks(a.size, chunk_bytes)
    dirty = np.zeros(nc, dtype=np.uint8)
    idx = np.zeros(nc, dtype=np.uint32)
    n = np.zeros(1, dtype=np.uint32)
    _check(_load().wmo_dirty_diff(_ptr(a), _ptr(p), a.size, chunk_bytes, _ptr(dirty), _ptr(idx), _ptr(n)),
           "dirty_diff")
    return dirty, idx[: int(n[0])].copy()


def encode(cache, chunk_bytes: int, dirty=None, crc_in=None, wire_cap: int | None = None, zero_tiles: bool = False,
           entropy: bool = False, ent_only: bool = False):
    """Return (wire u8[wire_len or wire_cap], crc u32[n_chunks], Result).  ``zero_tiles``: the
    option that ships a full tile of all-zero bytes as a table entry without payload.
    ``entropy``: the option that codes the exponents with the fixed prefix code (ENT tiles) where
    that is shorter than the bit planes.  ``ent_only`` (this oracle alone, for pinning the ENT coder):
    with ``entropy``, never choose a PACK tile."""
    b = _bytes_view(cache)
    nc = num_chunks(b.size, chunk_bytes)
    cap = wire_bound(b.size, chunk_bytes) if wire_cap is None else int(wire_cap)
    wire = np.zeros(cap, dtype=np.uint8)
    crc = np.zeros(nc, dtype=np.uint32) if crc_in is None else np.array(crc_in, dtype=np.uint32).copy()
    d = None if dirty is None else np.ascontiguousarray(dirty, dtype=np.uint8)
    res = _CResult()
    st = _load().wmo_encode_opt(_ptr(b), b.size, chunk_bytes, None if d is None else _ptr(d), _ptr(crc),
                                _ptr(wire), cap, (1 if zero_tiles else 0) | (2 if entropy else 0) | (4 if ent_only else 0), ctypes.byref(res))
    _check(st, "encode")
    r = _result(res)
    if r.status == 0:
        wire = wire[: r.wire_len].copy()
    return wire, crc, r


def decode_verify(wire, nbytes: int, chunk_bytes: int, dst=None, dst_crc=None, wire_len: int | None = None,
                  expect_entropy: bool | None = None):
    """Return (dst u8[nbytes], dst_crc u32[n_chunks], Result).  ``dst`` and ``dst_crc`` are
    copied first, so the caller's arrays play the part of the live state and stay untouched.
    ``expect_entropy``: None accepts images with and without ENT tiles; True / False is a receiver
    that knows the sender's option and refuses the other kind as a format error."""
    w = _bytes_view(wire)
    nc = num_chunks(nbytes, chunk_bytes)
    out = np.zeros(nbytes, dtype=np.uint8) if dst is None else _bytes_view(dst).copy()
    crc = np.zeros(nc, dtype=np.uint32) if dst_crc is None else np.array(dst_crc, dtype=np.uint32).copy()
    res = _CResult()
    st = _load().wmo_decode_verify_opt(_ptr(w), w.size if wire_len is None else int(wire_len), _ptr(out),
                                       nbytes, chunk_bytes, _ptr(crc),
                                       -1 if expect_entropy is None else int(bool(expect_entropy)), ctypes.byref(res))
    _check(st, "decode_verify")
    return out, crc, _result(res)


def flatten_leaves(leaves) -> np.ndarray:
    """The logical cache of the leaf-mode calls: the leaves' bytes one after the other."""
    return np.concatenate([_bytes_view(x) for x in leaves]) if len(leaves) else np.zeros(0, dtype=np.uint8)


def encode_leaves(leaves, chunk_bytes: int, dirty=None, crc_in=None, wire_cap: int | None = None,
                  zero_tiles: bool = False):
    """Leaf mode is defined by the flat calls: the image of a list of leaves is the image of their
    concatenation.  Returns what encode() returns."""
    return encode(flatten_leaves(leaves), chunk_bytes, dirty=dirty, crc_in=crc_in, wire_cap=wire_cap,
                  zero_tiles=zero_tiles)


def decode_verify_leaves(wire, leaves, chunk_bytes: int, dst_crc=None, wire_len: int | None = None):
    """Decode into a list of leaves (arrays whose sizes give the split).  Returns (new leaves,
    crc vector, Result); on failure the leaves come back as the flat decoder left its buffer."""
    sizes = [_bytes_view(x).size for x in leaves]
    flat = flatten_leaves(leaves)
    out, crc, res = decode_verify(wire, flat.size, chunk_bytes, dst=flat, dst_crc=dst_crc, wire_len=wire_len)
    parts, o = [], 0
    for n in sizes:
        parts.append(out[o:o + n].copy())
        o += n
    return parts, crc, res


def decode_verify_strict(wire, nbytes: int, chunk_bytes: int, dst, dst_crc, wire_len: int | None = None):
    """Verify first, write afterwards: what decode_verify returns when it succeeds; on any failure
    the destination and its CRC vector come back exactly as they were given."""
    out, crc, res = decode_verify(wire, nbytes, chunk_bytes, dst=dst, dst_crc=dst_crc, wire_len=wire_len)
    if res.status != 0:
        return _bytes_view(dst).copy(), np.array(dst_crc, dtype=np.uint32).copy(), res
    return out, crc, res
