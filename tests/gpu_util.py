"""Helpers for the GPU parity tests: run the C ABI through the Python binding on device
tensors and bring the outputs back as numpy arrays for comparison with the oracle."""
import numpy as np
import torch

from paper_2607_10389_b200 import binding as wm


def to_dev(a):
    if isinstance(a, torch.Tensor):
        return a.cuda()
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


class Gpu:
    """One geometry (nbytes, chunk_bytes) with its scratch buffers."""

    def __init__(self, nbytes, chunk_bytes):
        self.nbytes, self.chunk = nbytes, chunk_bytes
        self.nc = wm.num_chunks(nbytes, chunk_bytes)
        self.ws = wm.new_workspace(nbytes, chunk_bytes)
        self.res = wm.new_result()

    def checksum(self, cache):
        crc = torch.zeros(self.nc, dtype=torch.int32, device="cuda")
        wm.wm_checksum(cache, self.chunk, crc, self.ws)
        return crc.cpu().numpy().view(np.uint32)

    def dirty_diff(self, cache, prev, want_idx=True):
        dirty = torch.full((self.nc,), 7, dtype=torch.uint8, device="cuda")
        idx = torch.full((self.nc,), -1, dtype=torch.int32, device="cuda") if want_idx else None
        n = torch.zeros(1, dtype=torch.int32, device="cuda")
        wm.wm_dirty_diff(cache, prev, self.chunk, dirty, idx, n, self.ws)
        n = int(n.item())
        return dirty.cpu().numpy(), (idx.cpu().numpy().view(np.uint32)[:n] if want_idx else None), n

    def encode(self, cache, dirty=None, crc_in=None, wire_cap=None, canary=64):
        cap = wm.wire_bound(self.nbytes, self.chunk) if wire_cap is None else wire_cap
        wire = torch.full((cap + canary,), 0xA5, dtype=torch.uint8, device="cuda")
        crc = torch.zeros(self.nc, dtype=torch.int32, device="cuda") if crc_in is None else \
            torch.from_numpy(np.asarray(crc_in, dtype=np.uint32).view(np.int32).copy()).cuda()
        d = None if dirty is None else to_dev(np.asarray(dirty, dtype=np.uint8))
        wm.wm_encode(cache, self.chunk, d, crc, wire, self.ws, self.res, wire_cap=cap)
        r = wm.read_result(self.res)
        w = wire.cpu().numpy()
        assert (w[cap:] == 0xA5).all(), "encoder wrote past wire_cap"
        return w[:cap], crc.cpu().numpy().view(np.uint32), r, wire

    def decode(self, wire_dev, wire_len, dst=None, dst_crc=None):
        dst_t = torch.zeros(self.nbytes, dtype=torch.uint8, device="cuda") if dst is None else to_dev(dst).clone()
        crc = torch.zeros(self.nc, dtype=torch.int32, device="cuda") if dst_crc is None else \
            torch.from_numpy(np.asarray(dst_crc, dtype=np.uint32).view(np.int32).copy()).cuda()
        wm.wm_decode_verify(wire_dev, wire_len, dst_t, self.chunk, crc, self.ws, self.res)
        r = wm.read_result(self.res)
        return dst_t.cpu().numpy(), crc.cpu().numpy().view(np.uint32), r


def same_result(a, b):
    """Compare a binding Result with an oracle Result field by field."""
    return (a.status, a.first_bad_chunk, a.n_bad_chunks, a.n_present, a.wire_len, a.payload_bytes, a.cache_crc) == \
        (b.status, b.first_bad_chunk, b.n_bad_chunks, b.n_present, b.wire_len, b.payload_bytes, b.cache_crc)
