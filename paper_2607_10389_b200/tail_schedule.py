"""Verification placement on one GPU: the move is cut into super-chunks that travel separately.

The paper's verification-placement result (Section "Verification placement", the overlapped and
tail schedules) is that the checksum of a chunk can run while the following chunks are still on
the wire, so that only the last chunk's verification is exposed after the last byte arrives.
Restated on one GPU: the cache is cut into super-chunks (64 MiB by default, a whole number of
checksum chunks each), every super-chunk is a wire image of its own, and three streams carry

    encode(s)  ->  wire copy(s)  ->  decode + verify(s)

with a device-to-device copy standing in for the wire.  Super-chunk s is verified while s+1 is
copied and s+2 is encoded; after the last copy ends, one super-chunk's decode + verify is all
that remains.

This module only schedules calls of the C ABI (streams, events, one small pinned read of each
encode result for the image length a sender needs anyway); all arithmetic is in the library.
"""
from __future__ import annotations

import struct
from dataclasses import dataclass

import torch

from . import binding as wm

ALIGN = 256


@dataclass(frozen=True)
class Part:
    index: int
    offset: int          # bytes from the start of the cache
    nbytes: int
    first_chunk: int
    n_chunks: int
    wire_offset: int     # bytes from the start of each wire buffer
    wire_cap: int


def plan_parts(nbytes: int, chunk_bytes: int, super_bytes: int) -> list[Part]:
    """Cut [0, nbytes) into super-chunks of `super_bytes` (the last one may be shorter).

    `super_bytes` must be a positive multiple of `chunk_bytes`, so that every checksum chunk lies
    in exactly one part and the parts' chunk CRCs concatenate to the whole cache's.
    """
    if nbytes <= 0 or chunk_bytes <= 0 or super_bytes <= 0 or super_bytes % chunk_bytes:
        raise wm.WmError("super_bytes must be a positive multiple of chunk_bytes")
    parts, off, woff = [], 0, 0
    while off < nbytes:
        n = min(super_bytes, nbytes - off)
        cap = wm.wire_bound(n, chunk_bytes)
        parts.append(Part(len(parts), off, n, off // chunk_bytes, -(-n // chunk_bytes), woff, cap))
        off += n
        woff += -(-cap // ALIGN) * ALIGN
    return parts


def _parse(raw: bytes) -> wm.Result:
    st, fb, nb, npres, wl, pb, cc, _ = struct.unpack("<iIIIQQII", raw)
    return wm.Result(st, fb, nb, npres, wl, pb, cc)


@dataclass
class MoveReport:
    encode: list          # one Result per part
    decode: list          # one Result per part
    total_ms: float       # first encode starts -> last verification ends
    exposed_ms: float     # last wire copy ends -> last verification ends
    wire_bytes: int

    @property
    def ok(self) -> bool:
        return all(r.ok for r in self.encode) and all(r.ok for r in self.decode)


class TailSchedule:
    """Buffers, streams and events for moving one cache geometry super-chunk by super-chunk."""

    def __init__(self, nbytes: int, chunk_bytes: int, super_bytes: int = 64 << 20, device="cuda", strict=False,
                 ahead: int = 2, entropy: bool = False):
        self.nbytes, self.chunk_bytes, self.super_bytes = int(nbytes), int(chunk_bytes), int(super_bytes)
        self.parts = plan_parts(self.nbytes, self.chunk_bytes, self.super_bytes)
        self.strict = strict
        self.enc_options = wm.OPT_ENTROPY if entropy else 0
        self.dec_options = self.enc_options | (wm.OPT_STRICT if strict else 0)
        total_wire = self.parts[-1].wire_offset + self.parts[-1].wire_cap
        self.wire_send = torch.empty(total_wire, dtype=torch.uint8, device=device)
        self.wire_recv = torch.empty(total_wire, dtype=torch.uint8, device=device)
        big = max(p.nbytes for p in self.parts)
        self.ws_enc = wm.new_workspace(big, self.chunk_bytes, device)
        self.ws_dec = wm.new_workspace(big, self.chunk_bytes, device)
        n = len(self.parts)
        self.res_enc = torch.zeros((n, wm.RESULT_BYTES), dtype=torch.uint8, device=device)
        self.res_dec = torch.zeros((n, wm.RESULT_BYTES), dtype=torch.uint8, device=device)
        self.host_enc = torch.zeros((n, wm.RESULT_BYTES), dtype=torch.uint8).pin_memory()
        # arrived data is drained before new data is produced: the receiving side runs at high priority
        self.s_enc = torch.cuda.Stream(device=device)
        self.s_wire = torch.cuda.Stream(device=device, priority=-1)
        self.s_dec = torch.cuda.Stream(device=device, priority=-1)
        self.ev_enc = [torch.cuda.Event() for _ in range(n)]
        self.ev_wire = [torch.cuda.Event(enable_timing=(i == n - 1)) for i in range(n)]
        self.ev_start = torch.cuda.Event(enable_timing=True)
        self.ev_end = torch.cuda.Event(enable_timing=True)
        self._send = [self.wire_send[p.wire_offset: p.wire_offset + p.wire_cap] for p in self.parts]
        self._recv = [self.wire_recv[p.wire_offset: p.wire_offset + p.wire_cap] for p in self.parts]
        self._res_enc = [self.res_enc[i] for i in range(n)]
        self._res_dec = [self.res_dec[i] for i in range(n)]
        self._host_enc = [self.host_enc[i] for i in range(n)]
        self._host_np = self.host_enc.numpy()
        self.ahead = max(1, int(ahead))
        self.launches = 0

    def move(self, src: torch.Tensor, dst: torch.Tensor, src_crc: torch.Tensor, dst_crc: torch.Tensor,
             tamper=None) -> MoveReport:
        """Move `src` into `dst` part by part.  `src_crc` receives the source's chunk CRCs, `dst_crc`
        is updated for every part that verified.  `tamper(part, received_image)` may alter a part's
        received bytes before they are decoded (tests use it to damage one part on the wire)."""
        src, dst = src.reshape(-1).view(torch.uint8), dst.reshape(-1).view(torch.uint8)
        if src.numel() != self.nbytes or dst.numel() != self.nbytes:
            raise wm.WmError("cache size differs from the schedule's geometry")
        cur = torch.cuda.current_stream()
        for s in (self.s_enc, self.s_wire, self.s_dec):
            s.wait_stream(cur)
        C, n, launches = self.chunk_bytes, len(self.parts), 0
        enc, wire_bytes = [None] * n, 0
        self.ev_start.record(self.s_enc)
        # software pipeline on the host as well: encodes are issued `ahead` parts in front of the
        # part whose image length is read back, so that no stream waits for the issuing thread
        for i in range(n + self.ahead):
            if i < n:
                p = self.parts[i]
                wm.wm_encode_opt(src[p.offset: p.offset + p.nbytes], C, None,
                                 src_crc[p.first_chunk: p.first_chunk + p.n_chunks], self._send[i],
                                 self.ws_enc, self._res_enc[i], self.enc_options, stream=self.s_enc)
                launches += wm.last_launch_count()
                with torch.cuda.stream(self.s_enc):
                    self._host_enc[i].copy_(self._res_enc[i], non_blocking=True)
                self.ev_enc[i].record(self.s_enc)
            j = i - self.ahead
            if j < 0:
                continue
            p = self.parts[j]
            self.ev_enc[j].synchronize()                   # the sender learns the image length
            r = _parse(self._host_np[j].tobytes())
            enc[j] = r
            length = r.wire_len if r.ok else 0
            wire_bytes += length
            if length:
                with torch.cuda.stream(self.s_wire):
                    self._recv[j][:length].copy_(self._send[j][:length], non_blocking=True)
                    if tamper is not None:
                        tamper(p, self._recv[j][:length])
            self.ev_wire[j].record(self.s_wire)
            self.s_dec.wait_event(self.ev_wire[j])
            wm.wm_decode_verify_opt(self._recv[j], length, dst[p.offset: p.offset + p.nbytes], C,
                                    dst_crc[p.first_chunk: p.first_chunk + p.n_chunks], self.ws_dec, self._res_dec[j],
                                    self.dec_options, stream=self.s_dec)
            launches += wm.last_launch_count()
        self.ev_end.record(self.s_dec)
        cur.wait_stream(self.s_dec)
        self.ev_end.synchronize()
        self.launches = launches
        raw = self.res_dec.cpu().numpy()
        dec = [_parse(raw[i].tobytes()) for i in range(len(self.parts))]
        return MoveReport(enc, dec, self.ev_start.elapsed_time(self.ev_end),
                          self.ev_wire[-1].elapsed_time(self.ev_end), wire_bytes)
