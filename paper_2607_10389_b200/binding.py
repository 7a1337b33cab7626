"""Thin Python binding of the C ABI in ``include/wm.h`` (argument marshalling only).

Every step of the path runs in the CUDA library; torch is used for device memory and
streams.  There is no CPU fallback: importing this module without the built library, or
calling it without a CUDA device, raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libwm.so")

STATUS = {
    0: "OK", -1: "ERR_ARG", -2: "ERR_CAPACITY", -3: "ERR_FORMAT", -4: "ERR_META_CRC", -5: "ERR_STRUCT",
    -6: "ERR_DESC", -7: "ERR_CHUNK_CRC", -8: "ERR_STALE", -9: "ERR_CACHE_CRC", -10: "ERR_TIMEOUT",
    -11: "ERR_CUDA",
}
RESULT_BYTES = 40
EXPORTS = ("wm_num_chunks", "wm_num_tiles", "wm_meta_bytes", "wm_wire_bound", "wm_workspace_bytes",
           "wm_checksum", "wm_dirty_diff", "wm_encode", "wm_decode_verify", "wm_last_launch_count",
           "wm_timing_enable", "wm_timing_read_ms", "wm_checksum_noalloc", "wm_encode_leaves",
           "wm_decode_verify_leaves", "wm_zero_tiles_enable", "wm_decode_verify_strict", "wm_checksum_poly", "wm_entropy_enable",
           "wm_encode_opt", "wm_decode_verify_opt", "wm_checksum_xxh64", "wm_wait_budget_ms", "wm_workspace_status",
           "wm_inject_stall")


class WmError(RuntimeError):
    pass


def load_library() -> ctypes.CDLL:
    if not os.path.exists(_SO):
        raise WmError(f"{_SO} is missing: build it with `python -m paper_2607_10389_b200.build` "
                      "(there is no CPU fallback)")
    lib = ctypes.CDLL(_SO)
    u64, u32, vp = ctypes.c_uint64, ctypes.c_uint32, ctypes.c_void_p
    lib.wm_num_chunks.restype = u64
    lib.wm_num_chunks.argtypes = [u64, u32]
    lib.wm_num_tiles.restype = u64
    lib.wm_num_tiles.argtypes = [u64]
    for n in ("wm_meta_bytes", "wm_wire_bound", "wm_workspace_bytes"):
        getattr(lib, n).restype = u64
        getattr(lib, n).argtypes = [u64, u32]
    lib.wm_last_launch_count.restype = u32
    lib.wm_last_launch_count.argtypes = []
    lib.wm_timing_enable.restype = None
    lib.wm_timing_enable.argtypes = [ctypes.c_int]
    lib.wm_zero_tiles_enable.restype = None
    lib.wm_zero_tiles_enable.argtypes = [ctypes.c_int]
    lib.wm_entropy_enable.restype = None
    lib.wm_entropy_enable.argtypes = [ctypes.c_int]
    lib.wm_wait_budget_ms.restype = None
    lib.wm_wait_budget_ms.argtypes = [u32]
    lib.wm_inject_stall.restype = None
    lib.wm_inject_stall.argtypes = [ctypes.c_int]
    lib.wm_workspace_status.restype = ctypes.c_int
    lib.wm_workspace_status.argtypes = [vp, vp]
    lib.wm_timing_read_ms.restype = ctypes.c_int
    lib.wm_timing_read_ms.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_float)]
    lib.wm_checksum.restype = ctypes.c_int
    lib.wm_checksum.argtypes = [vp, u64, u32, vp, vp, u64, vp]
    lib.wm_checksum_poly.restype = ctypes.c_int
    lib.wm_checksum_poly.argtypes = [vp, u64, u32, ctypes.c_int, vp, vp, u64, vp]
    lib.wm_checksum_xxh64.restype = ctypes.c_int
    lib.wm_checksum_xxh64.argtypes = [vp, u64, u32, u64, vp, vp]
    lib.wm_checksum_noalloc.restype = ctypes.c_int
    lib.wm_checksum_noalloc.argtypes = [vp, u64, u32, vp, vp]
    lib.wm_dirty_diff.restype = ctypes.c_int
    lib.wm_dirty_diff.argtypes = [vp, vp, u64, u32, vp, vp, vp, vp, u64, vp]
    lib.wm_encode.restype = ctypes.c_int
    lib.wm_encode.argtypes = [vp, u64, u32, vp, vp, vp, u64, vp, u64, vp, vp]
    lib.wm_decode_verify.restype = ctypes.c_int
    lib.wm_decode_verify.argtypes = [vp, u64, vp, u64, u32, vp, vp, u64, vp, vp]
    lib.wm_decode_verify_strict.restype = ctypes.c_int
    lib.wm_decode_verify_strict.argtypes = [vp, u64, vp, u64, u32, vp, vp, u64, vp, vp]
    lib.wm_encode_opt.restype = ctypes.c_int
    lib.wm_encode_opt.argtypes = [vp, vp, u32, u64, u32, vp, vp, vp, u64, vp, u64, u32, vp, vp]
    lib.wm_decode_verify_opt.restype = ctypes.c_int
    lib.wm_decode_verify_opt.argtypes = [vp, u64, vp, vp, u32, u64, u32, vp, vp, u64, u32, vp, vp]
    lib.wm_encode_leaves.restype = ctypes.c_int
    lib.wm_encode_leaves.argtypes = [vp, u32, u64, u32, vp, vp, vp, u64, vp, u64, vp, vp]
    lib.wm_decode_verify_leaves.restype = ctypes.c_int
    lib.wm_decode_verify_leaves.argtypes = [vp, u64, vp, u32, u64, u32, vp, vp, u64, vp, vp]
    return lib


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = load_library()
    return _lib


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

    @property
    def ok(self) -> bool:
        return self.status == 0


def read_result(result_dev: torch.Tensor) -> Result:
    """Copy a 40-byte device result record to the host (synchronises the current stream)."""
    raw = result_dev.cpu().numpy().tobytes()
    import struct
    st, fb, nb, npres, wl, pb, cc, _ = struct.unpack("<iIIIQQII", raw)
    return Result(st, fb, nb, npres, wl, pb, cc)


def num_chunks(nbytes: int, chunk_bytes: int) -> int:
    return int(lib().wm_num_chunks(nbytes, chunk_bytes))


def num_tiles(nbytes: int) -> int:
    return int(lib().wm_num_tiles(nbytes))


def meta_bytes(nbytes: int, chunk_bytes: int) -> int:
    return int(lib().wm_meta_bytes(nbytes, chunk_bytes))


def wire_bound(nbytes: int, chunk_bytes: int) -> int:
    return int(lib().wm_wire_bound(nbytes, chunk_bytes))


def workspace_bytes(nbytes: int, chunk_bytes: int) -> int:
    return int(lib().wm_workspace_bytes(nbytes, chunk_bytes))


def last_launch_count() -> int:
    return int(lib().wm_last_launch_count())


KIND_CHECKSUM, KIND_DIFF, KIND_ENCODE, KIND_DECODE = 0, 1, 2, 3


def timing_enable(on: bool) -> None:
    lib().wm_timing_enable(1 if on else 0)


def zero_tiles_enable(on: bool) -> None:
    """Encoder option: full tiles of all-zero bytes become table entries without payload."""
    lib().wm_zero_tiles_enable(1 if on else 0)


def entropy_enable(on: bool) -> None:
    """Codec option: entropy-coded exponents (ENT tiles).  Applies to the encode calls (what they
    write) and to the decode calls (what they expect) of this process."""
    lib().wm_entropy_enable(1 if on else 0)


def wait_budget_ms(ms: int) -> None:
    """Upper bound of every device-side wait of the calls issued from now on (default 2000 ms)."""
    lib().wm_wait_budget_ms(int(ms))


def inject_stall(on: bool) -> None:
    """Test hook: calls issued while it is on leave out what their bounded waits wait for, so the
    waits run out after the budget and the calls end in ERR_TIMEOUT."""
    lib().wm_inject_stall(1 if on else 0)


def workspace_status(workspace, stream=None) -> int:
    """Device-side outcome (a wm_status) of the last call that used `workspace` on the stream;
    None stands for the built-in scratch of wm_checksum_noalloc.  Synchronises the stream."""
    return int(lib().wm_workspace_status(None if workspace is None else workspace.data_ptr(), _stream(stream)))


def timing_read_ms(kind: int) -> float:
    ms = ctypes.c_float(0.0)
    _check(lib().wm_timing_read_ms(kind, ctypes.byref(ms)), "wm_timing_read_ms")
    return float(ms.value)


def _dev_u8(t: torch.Tensor, what: str) -> torch.Tensor:
    if not t.is_cuda:
        raise WmError(f"{what} must be a CUDA tensor (there is no CPU path)")
    if not t.is_contiguous():
        raise WmError(f"{what} must be contiguous")
    return t


def _stream(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise WmError(f"{what}: {STATUS.get(rc, rc)}")


def new_workspace(nbytes: int, chunk_bytes: int, device="cuda") -> torch.Tensor:
    n = workspace_bytes(nbytes, chunk_bytes)
    if n == 0:
        raise WmError("bad geometry")
    return torch.empty(n, dtype=torch.uint8, device=device)


def new_result(device="cuda") -> torch.Tensor:
    return torch.zeros(RESULT_BYTES, dtype=torch.uint8, device=device)


def wm_checksum(cache: torch.Tensor, chunk_bytes: int, crc_out: torch.Tensor, workspace: torch.Tensor,
                stream=None) -> None:
    _dev_u8(cache, "cache")
    nbytes = cache.numel() * cache.element_size()
    _check(lib().wm_checksum(cache.data_ptr(), nbytes, chunk_bytes, crc_out.data_ptr(), workspace.data_ptr(),
                             workspace.numel(), _stream(stream)), "wm_checksum")


POLY_CRC32C, POLY_ZLIB = 0, 1


def wm_checksum_poly(cache: torch.Tensor, chunk_bytes: int, polynomial: int, crc_out: torch.Tensor,
                     workspace: torch.Tensor, stream=None) -> None:
    """wm_checksum with the polynomial chosen by the caller (POLY_CRC32C or POLY_ZLIB)."""
    _dev_u8(cache, "cache")
    nbytes = cache.numel() * cache.element_size()
    _check(lib().wm_checksum_poly(cache.data_ptr(), nbytes, chunk_bytes, int(polynomial), crc_out.data_ptr(),
                                  workspace.data_ptr(), workspace.numel(), _stream(stream)), "wm_checksum_poly")


def wm_checksum_xxh64(cache: torch.Tensor, chunk_bytes: int, seed: int, hash_out: torch.Tensor, stream=None) -> None:
    """XXH64 of every chunk into an int64 / uint64 tensor of n_chunks entries."""
    _dev_u8(cache, "cache")
    nbytes = cache.numel() * cache.element_size()
    _check(lib().wm_checksum_xxh64(cache.data_ptr(), nbytes, chunk_bytes, int(seed) & 0xFFFFFFFFFFFFFFFF, hash_out.data_ptr(),
                                   _stream(stream)), "wm_checksum_xxh64")


NOALLOC_MAX_BYTES = 4 << 30


def wm_checksum_noalloc(cache: torch.Tensor, chunk_bytes: int, crc_out: torch.Tensor, stream=None,
                        nbytes: int | None = None) -> None:
    """wm_checksum without a workspace argument: scratch and tables are built into the library,
    for callers that may not allocate device memory.  `nbytes` overrides the tensor's size
    (used to exercise the size limit without allocating a buffer that large)."""
    _dev_u8(cache, "cache")
    n = cache.numel() * cache.element_size() if nbytes is None else int(nbytes)
    _check(lib().wm_checksum_noalloc(cache.data_ptr(), n, chunk_bytes, crc_out.data_ptr(), _stream(stream)),
           "wm_checksum_noalloc")


def wm_dirty_diff(cache: torch.Tensor, prev: torch.Tensor, chunk_bytes: int, dirty_out: torch.Tensor,
                  dirty_idx_out, n_dirty_out: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
    _dev_u8(cache, "cache")
    _dev_u8(prev, "prev")
    nbytes = cache.numel() * cache.element_size()
    if prev.numel() * prev.element_size() != nbytes:
        raise WmError("snapshots differ in size")
    _check(lib().wm_dirty_diff(cache.data_ptr(), prev.data_ptr(), nbytes, chunk_bytes, dirty_out.data_ptr(),
                               None if dirty_idx_out is None else dirty_idx_out.data_ptr(),
                               n_dirty_out.data_ptr(), workspace.data_ptr(), workspace.numel(),
                               _stream(stream)), "wm_dirty_diff")


def wm_encode(cache: torch.Tensor, chunk_bytes: int, dirty, crc_inout: torch.Tensor, wire: torch.Tensor,
              workspace: torch.Tensor, result: torch.Tensor, stream=None, wire_cap=None) -> None:
    _dev_u8(cache, "cache")
    _dev_u8(wire, "wire")
    nbytes = cache.numel() * cache.element_size()
    cap = wire.numel() if wire_cap is None else int(wire_cap)
    _check(lib().wm_encode(cache.data_ptr(), nbytes, chunk_bytes, None if dirty is None else dirty.data_ptr(),
                           crc_inout.data_ptr(), wire.data_ptr(), cap, workspace.data_ptr(), workspace.numel(),
                           result.data_ptr(), _stream(stream)), "wm_encode")


def wm_decode_verify(wire: torch.Tensor, wire_len: int, dst: torch.Tensor, chunk_bytes: int,
                     dst_crc_inout: torch.Tensor, workspace: torch.Tensor, result: torch.Tensor,
                     stream=None) -> None:
    _dev_u8(wire, "wire")
    _dev_u8(dst, "dst")
    nbytes = dst.numel() * dst.element_size()
    _check(lib().wm_decode_verify(wire.data_ptr(), int(wire_len), dst.data_ptr(), nbytes, chunk_bytes,
                                  dst_crc_inout.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                  result.data_ptr(), _stream(stream)), "wm_decode_verify")


def wm_decode_verify_strict(wire: torch.Tensor, wire_len: int, dst: torch.Tensor, chunk_bytes: int,
                            dst_crc_inout: torch.Tensor, workspace: torch.Tensor, result: torch.Tensor,
                            stream=None) -> None:
    """wm_decode_verify that stores nothing until every check has passed."""
    _dev_u8(wire, "wire")
    _dev_u8(dst, "dst")
    nbytes = dst.numel() * dst.element_size()
    _check(lib().wm_decode_verify_strict(wire.data_ptr(), int(wire_len), dst.data_ptr(), nbytes, chunk_bytes,
                                         dst_crc_inout.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                         result.data_ptr(), _stream(stream)), "wm_decode_verify_strict")


OPT_ZERO_TILES, OPT_ENTROPY, OPT_STRICT = 1, 2, 4


def opt_blocks(n: int) -> int:
    """Option bits that cap the main kernel at n thread blocks (each takes one SM); 0: no cap."""
    return (int(n) & 0xFF) << 8



def wm_encode_opt(cache, chunk_bytes: int, dirty, crc_inout: torch.Tensor, wire: torch.Tensor, workspace: torch.Tensor,
                  result: torch.Tensor, options: int, stream=None, leaf_table=None, nbytes=None) -> None:
    """wm_encode / wm_encode_leaves with the options given per call (OPT_ZERO_TILES, OPT_ENTROPY).
    Flat form: `cache` is a tensor; leaf form: `cache` is None, `leaf_table` and `nbytes` are given."""
    _dev_u8(wire, "wire")
    if leaf_table is None:
        _dev_u8(cache, "cache")
        n, cp, lp, nl = cache.numel() * cache.element_size(), cache.data_ptr(), None, 0
    else:
        n, cp, lp, nl = int(nbytes), None, leaf_table.data_ptr(), leaf_table.shape[0]
    _check(lib().wm_encode_opt(cp, lp, nl, n, chunk_bytes, None if dirty is None else dirty.data_ptr(), crc_inout.data_ptr(),
                               wire.data_ptr(), wire.numel(), workspace.data_ptr(), workspace.numel(), int(options),
                               result.data_ptr(), _stream(stream)), "wm_encode_opt")


def wm_decode_verify_opt(wire: torch.Tensor, wire_len: int, dst, chunk_bytes: int, dst_crc_inout: torch.Tensor,
                         workspace: torch.Tensor, result: torch.Tensor, options: int, stream=None, leaf_table=None,
                         nbytes=None) -> None:
    """The decode calls with the options given per call (OPT_ENTROPY: the image holds ENT tiles;
    OPT_STRICT: nothing is stored before the verdict)."""
    _dev_u8(wire, "wire")
    if leaf_table is None:
        _dev_u8(dst, "dst")
        n, dp, lp, nl = dst.numel() * dst.element_size(), dst.data_ptr(), None, 0
    else:
        n, dp, lp, nl = int(nbytes), None, leaf_table.data_ptr(), leaf_table.shape[0]
    _check(lib().wm_decode_verify_opt(wire.data_ptr(), int(wire_len), dp, lp, nl, n, chunk_bytes, dst_crc_inout.data_ptr(),
                                      workspace.data_ptr(), workspace.numel(), int(options), result.data_ptr(),
                                      _stream(stream)), "wm_decode_verify_opt")


def make_leaf_table(tensors, device="cuda") -> torch.Tensor:
    """Device table of (ptr, nbytes) pairs, one per tensor, in the order given: the `wm_leaf`
    array of the leaf-mode calls.  The tensors must stay alive while the table is in use."""
    rows = []
    for t in tensors:
        if not t.is_cuda or not t.is_contiguous():
            raise WmError("leaves must be contiguous CUDA tensors")
        rows.append((t.data_ptr(), t.numel() * t.element_size()))
    table = torch.tensor(rows, dtype=torch.int64).reshape(-1, 2)
    return table.to(device)


def wm_encode_leaves(leaf_table: torch.Tensor, nbytes: int, chunk_bytes: int, dirty, crc_inout: torch.Tensor,
                     wire: torch.Tensor, workspace: torch.Tensor, result: torch.Tensor, stream=None,
                     wire_cap=None) -> None:
    _dev_u8(wire, "wire")
    cap = wire.numel() if wire_cap is None else int(wire_cap)
    _check(lib().wm_encode_leaves(leaf_table.data_ptr(), leaf_table.shape[0], int(nbytes), chunk_bytes,
                                  None if dirty is None else dirty.data_ptr(), crc_inout.data_ptr(), wire.data_ptr(),
                                  cap, workspace.data_ptr(), workspace.numel(), result.data_ptr(), _stream(stream)),
           "wm_encode_leaves")


def wm_decode_verify_leaves(wire: torch.Tensor, wire_len: int, leaf_table: torch.Tensor, nbytes: int,
                            chunk_bytes: int, dst_crc_inout: torch.Tensor, workspace: torch.Tensor,
                            result: torch.Tensor, stream=None) -> None:
    _dev_u8(wire, "wire")
    _check(lib().wm_decode_verify_leaves(wire.data_ptr(), int(wire_len), leaf_table.data_ptr(), leaf_table.shape[0],
                                         int(nbytes), chunk_bytes, dst_crc_inout.data_ptr(), workspace.data_ptr(),
                                         workspace.numel(), result.data_ptr(), _stream(stream)),
           "wm_decode_verify_leaves")
