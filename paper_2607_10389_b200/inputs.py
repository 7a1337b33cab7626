"""Seeded synthetic attention caches and dirty patterns.

This module only draws random numbers and lays them out; it holds none of the mover's
arithmetic (no checksum, no codec).  Both the CUDA tests/benchmark and the CPU oracle's
tests take their inputs from here, so the two sides always read the same bytes: data is
drawn once (on the device it is asked for) and copied, never drawn twice.

The caches stand in for the paper's warmed world-model cache (Section 3.1: 1.67 GB of bf16
attention KV; Section 6.4: 99.99 % bf16), which is not available: they take its dtype, size
and chunking, the dirty fraction of Section 3.3 / Appendix G (about three quarters of the
chunks rewritten per generation step), and value distributions chosen to look like
attention keys and values (Gaussian, with per-channel scales and a few outlier channels on
the key side).
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

TILE_BYTES = 16384


@dataclass(frozen=True)
class CacheConfig:
    name: str
    shape: tuple          # (layers, 2, kv_heads, tokens, head_dim); () for raw random bytes
    nbytes: int
    chunk_bytes: int
    seed: int
    kind: str             # "gauss" | "kv" | "bytes" | "llm"
    fill: float = 1.0     # "llm": fraction of the token window that holds data (the rest is zero)


def _kv(name, shape, chunk, seed, kind, fill=1.0):
    n = 2
    for s in shape:
        n *= s
    return CacheConfig(name, tuple(shape), n, chunk, seed, kind, fill)


CONFIGS = {
    # tiny cache, plain Gaussian
    "tiny": _kv("tiny", (4, 2, 8, 256, 64), 64 * 1024, 1, "gauss"),
    "tiny8m": _kv("tiny8m", (4, 2, 8, 1024, 64), 64 * 1024, 1, "gauss"),
    # engine-sized cache (the headline workload)
    "engine": _kv("engine", (30, 2, 16, 6800, 128), 1 << 20, 2, "kv"),
    # incompressible stress
    "random": CacheConfig("random", (), 1 << 30, 1 << 20, 3, "bytes"),
    # long-context cache
    "long": _kv("long", (32, 2, 8, 131072, 128), 4 << 20, 4, "kv"),
    "long8g": _kv("long8g", (32, 2, 8, 65536, 128), 4 << 20, 4, "kv"),
    # engine-like cache small enough for a profiler capture, still larger than the 126 MB L2
    "engine_256m": _kv("engine_256m", (5, 2, 16, 6400, 128), 1 << 20, 2, "kv"),
    # append-only text-model cache (Section 3.3: 24 layers, a window that fills from 0.249 towards
    # 0.727, a step appends tokens and rewrites nothing): allocated for the whole window, zero
    # beyond the tokens written so far
    "llm_append": _kv("llm_append", (24, 2, 8, 16384, 128), 64 * 1024, 6, "llm", 0.249),
    "llm_append_small": _kv("llm_append_small", (2, 2, 2, 2048, 128), 64 * 1024, 6, "llm", 0.249),
    # reduced engine-like cache for tests that also run the CPU oracle on everything
    "engine_small": _kv("engine_small", (3, 2, 4, 680, 128), 1 << 20, 2, "kv"),
}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def make_cache(cfg: CacheConfig, device="cpu", head_bytes: int | None = None) -> torch.Tensor:
    """Return the cache as a flat uint8 tensor of cfg.nbytes bytes on `device`.  With `head_bytes`
    only the leading layers that cover that many bytes are drawn (the same bytes the whole cache
    begins with: layers are drawn one after the other from one generator)."""
    device = torch.device(device)
    if head_bytes is not None and cfg.kind in ("kv", "gauss"):
        per_layer = cfg.nbytes // cfg.shape[0]
        keep = min(cfg.shape[0], -(-head_bytes // per_layer))
        head = CacheConfig(cfg.name, (keep,) + tuple(cfg.shape[1:]), keep * per_layer, cfg.chunk_bytes, cfg.seed, cfg.kind, cfg.fill)
        return make_cache(head, device)
    g = _gen(cfg.seed, device)
    if cfg.kind == "bytes":
        out = torch.empty(cfg.nbytes, dtype=torch.uint8, device=device)
        step = 1 << 28
        for o in range(0, cfg.nbytes, step):
            n = min(step, cfg.nbytes - o)
            out[o:o + n] = torch.randint(0, 256, (n,), generator=g, device=device, dtype=torch.uint8)
        return out
    layers, two, heads, tokens, dim = cfg.shape
    assert two == 2
    if cfg.kind == "llm":
        out = torch.zeros(cfg.shape, dtype=torch.bfloat16, device=device)
        filled = filled_tokens(cfg)
        for layer in range(layers):
            k = torch.randn((heads, filled, dim), generator=g, device=device)
            v = torch.randn((heads, filled, dim), generator=g, device=device)
            scale = torch.exp(0.5 * torch.randn((heads, 1, dim), generator=g, device=device))
            out[layer, 0, :, :filled] = (k * scale).to(torch.bfloat16)
            out[layer, 1, :, :filled] = v.to(torch.bfloat16)
        return out.view(-1).view(torch.uint8)
    out = torch.empty(cfg.shape, dtype=torch.bfloat16, device=device)
    for layer in range(layers):
        k = torch.randn((heads, tokens, dim), generator=g, device=device)
        v = torch.randn((heads, tokens, dim), generator=g, device=device)
        if cfg.kind == "kv":
            # keys: per-(head, channel) lognormal(0, 0.5) scale, 4 outlier channels per head x10
            scale = torch.exp(0.5 * torch.randn((heads, 1, dim), generator=g, device=device))
            for h in range(heads):
                ch = torch.randperm(dim, generator=g, device=device)[:4]
                scale[h, 0, ch] *= 10.0
            k = k * scale
        out[layer, 0] = k.to(torch.bfloat16)
        out[layer, 1] = v.to(torch.bfloat16)
        del k, v
    return out.view(-1).view(torch.uint8)


def fresh_like(cache_u8: torch.Tensor, seed: int, lo: int, hi: int) -> torch.Tensor:
    """Fresh Gaussian bf16 bytes for the byte range [lo, hi) of a cache (lo, hi even)."""
    g = _gen(seed, cache_u8.device)
    n = (hi - lo) // 2
    return torch.randn((n,), generator=g, device=cache_u8.device).to(torch.bfloat16).view(torch.uint8)


def rewrite_random_chunks(cache_u8: torch.Tensor, chunk_bytes: int, fraction: float, seed: int):
    """Second snapshot: a seeded random `fraction` of the chunks receives fresh draws.
    Returns (new_cache, rewritten u8[n_chunks])."""
    n = cache_u8.numel()
    nc = (n + chunk_bytes - 1) // chunk_bytes
    g = torch.Generator().manual_seed(seed)
    perm = torch.randperm(nc, generator=g)
    k = int(round(fraction * nc))
    mask = torch.zeros(nc, dtype=torch.uint8)
    mask[perm[:k]] = 1
    new = cache_u8.clone()
    for c in torch.nonzero(mask).flatten().tolist():
        lo, hi = c * chunk_bytes, min((c + 1) * chunk_bytes, n)
        new[lo:hi] = fresh_like(cache_u8, seed * 1000003 + c, lo, hi + ((hi - lo) & 1))[: hi - lo]
    return new, mask


def step_pattern(n_chunks: int, n_groups: int, fraction: float, seed: int) -> torch.Tensor:
    """Dirty pattern of one generation step: chunk indices are split into `n_groups`
    contiguous groups (one per layer); in each group a contiguous, wrapping run covering
    `fraction` of the group is rewritten, its start drawn from `seed`.  Mirrors the rolling
    window of Section 3.3 (each block overwrites part of the window)."""
    g = torch.Generator().manual_seed(seed)
    mask = torch.zeros(n_chunks, dtype=torch.uint8)
    bounds = [round(i * n_chunks / n_groups) for i in range(n_groups + 1)]
    for i in range(n_groups):
        lo, hi = bounds[i], bounds[i + 1]
        size = hi - lo
        if size <= 0:
            continue
        run = int(round(fraction * size))
        start = int(torch.randint(0, size, (1,), generator=g))
        for j in range(run):
            mask[lo + (start + j) % size] = 1
    return mask


def apply_step(cache_u8: torch.Tensor, chunk_bytes: int, mask: torch.Tensor, seed: int) -> None:
    """Rewrite, in place, every chunk flagged in `mask` with fresh draws."""
    n = cache_u8.numel()
    idx = torch.nonzero(mask).flatten().tolist()
    # contiguous runs are rewritten with one draw each
    i = 0
    while i < len(idx):
        j = i
        while j + 1 < len(idx) and idx[j + 1] == idx[j] + 1:
            j += 1
        lo, hi = idx[i] * chunk_bytes, min((idx[j] + 1) * chunk_bytes, n)
        cache_u8[lo:hi] = fresh_like(cache_u8, seed * 1000003 + idx[i], lo, hi + ((hi - lo) & 1))[: hi - lo]
        i = j + 1


def filled_tokens(cfg: CacheConfig) -> int:
    """Tokens of an "llm" cache's window that hold data."""
    return int(round(cfg.fill * cfg.shape[3]))


def before_append(cache_u8: torch.Tensor, cfg: CacheConfig, appended: int):
    """The previous snapshot of an append-only cache: the same bytes without the last `appended`
    tokens of every (layer, key/value, head) row block.  Returns (prev, dirty u8[n_chunks]): the
    chunks that hold those tokens are the only ones that differ."""
    layers, two, heads, tokens, dim = cfg.shape
    filled = filled_tokens(cfg)
    prev = cache_u8.clone()
    view = prev.view(torch.bfloat16).view(cfg.shape)
    view[:, :, :, filled - appended:filled] = 0
    nc = (cfg.nbytes + cfg.chunk_bytes - 1) // cfg.chunk_bytes
    mask = torch.zeros(nc, dtype=torch.uint8)
    row = dim * 2
    for blk in range(layers * two * heads):
        lo = (blk * tokens + filled - appended) * row
        hi = (blk * tokens + filled) * row
        mask[lo // cfg.chunk_bytes:(hi - 1) // cfg.chunk_bytes + 1] = 1
    return prev, mask


def append_schedule(cfg: CacheConfig, steps: int, fill_to: float = 0.727):
    """Token counts of an append-only run (Section 3.3: the window of the text model fills from
    0.249 towards 0.727 while no step rewrites anything): `steps` appends that take the window
    from cfg.fill to `fill_to` in equal parts, with one step in the middle that appends nothing
    (an all-clean step).  Returns a list of (first_token, count)."""
    first, last = filled_tokens(cfg), int(round(fill_to * cfg.shape[3]))
    real = steps - 1
    edges = [first + (last - first) * i // real for i in range(real + 1)]
    out = [(edges[i], edges[i + 1] - edges[i]) for i in range(real)]
    out.insert(real // 2, (edges[real // 2], 0))
    return out


def append_tokens(cache_u8: torch.Tensor, cfg: CacheConfig, first: int, count: int, seed: int) -> torch.Tensor:
    """Append `count` tokens at position `first` of every (layer, key/value, head) row block, in
    place, with fresh draws; nothing else is touched.  Returns the chunks that hold them (u8[n_chunks])."""
    layers, two, heads, tokens, dim = cfg.shape
    nc = (cfg.nbytes + cfg.chunk_bytes - 1) // cfg.chunk_bytes
    mask = torch.zeros(nc, dtype=torch.uint8)
    if count == 0:
        return mask
    g = _gen(seed, cache_u8.device)
    view = cache_u8.view(torch.bfloat16).view(cfg.shape)
    fresh = torch.randn((layers, two, heads, count, dim), generator=g, device=cache_u8.device)
    fresh = torch.where(fresh == 0, torch.ones_like(fresh), fresh)       # (a token written is never all zero bits)
    view[:, :, :, first:first + count] = fresh.to(torch.bfloat16)
    row = dim * 2
    for blk in range(layers * two * heads):
        lo = (blk * tokens + first) * row
        hi = (blk * tokens + first + count) * row
        mask[lo // cfg.chunk_bytes:(hi - 1) // cfg.chunk_bytes + 1] = 1
    return mask


PAPER_CACHE_BYTES = 1_670_124_960      # the movable set of the paper's engine (Section 6.3)


def paper_leaf_sizes(seed: int = 9, tensors: int = 420, flags: int = 30, total: int = PAPER_CACHE_BYTES):
    """Sizes (bytes) of a leaf table shaped like the paper's movable set (Section 3.1, Section 5:
    420 tensors, 450 manifest leaves with the scalar control flags; Section 6.3: 1,670,124,960
    bytes in all).  The tensors get seeded random sizes (multiples of 256 bytes, a factor of four
    between the smallest and the largest), the flags 2 to 64 bytes each, one flag after every
    fourteenth tensor; the last tensor takes what is left, so the sizes add up to `total`."""
    g = torch.Generator().manual_seed(seed)
    flag_sizes = [int(x) for x in (2 ** torch.randint(1, 7, (flags,), generator=g))]
    weights = 1.0 + 3.0 * torch.rand(tensors, generator=g)
    room = total - sum(flag_sizes)
    sizes = [int(room * float(w / weights.sum())) // 256 * 256 for w in weights]
    sizes[-1] = room - sum(sizes[:-1])
    assert min(sizes) > 0
    out, every = [], tensors // flags
    for i, n in enumerate(sizes):
        out.append(n)
        if (i + 1) % every == 0 and flag_sizes:
            out.append(flag_sizes.pop())
    assert sum(out) == total and len(out) == tensors + flags
    return out
