#!/usr/bin/env python
"""Benchmark of the session mover's data path on B200.

One "step" is one pass of the whole path over one synthetic cache that is already resident
in HBM: wm_checksum -> wm_dirty_diff (against a snapshot with three quarters of the chunks
rewritten) -> wm_encode (full move: fused checksum + encode) -> wm_decode_verify into a shadow
buffer.  `value` is raw cache bytes per second through that whole step; the per-call rates
(the metric's "checksum+encode" and "decode+verify" figures) are in `calls`.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload engine] [--impl reference]

N > 1 runs one independent replica per GPU (the path has no exchange step): launch with
torch.distributed.run; rank 0 prints the one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

FALLBACK_HBM_GBS = 6650.0
# DRAM bytes read + written per launch of the encode kernel, from single-pass ncu captures of this
# benchmark (dram__bytes_read.sum + dram__bytes_write.sum; summaries under profiles/).  A workload
# without a capture reports null.
NCU_TRAFFIC_BYTES = {"engine": 1671721728 + 1208218624, "engine_256m": 262455000 + 145051000}


# the headline metric as the baseline file words it; a step is one pass of the whole path:
# wm_checksum, wm_dirty_diff, wm_encode (full, fused with the checksum) and wm_decode_verify
L2_BYTES = 126 * 1000 * 1000          # B200 L2
L2_FLUSH_BYTES = 256 << 20
METRIC = "raw-cache GB/s for checksum+encode and decode+verify, % HBM roofline, ratio"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU through NVML while running."""

    def __init__(self, index: int, uuid: str | None = None, period_s: float = 0.01):
        self.index, self.uuid, self.period = index, uuid, period_s
        self.samples, self._stop, self._thread = [], threading.Event(), None
        self.max_mhz = None

    def _open(self):
        """NVML handle of the GPU (done before the timed region, so that even a region of a few
        milliseconds gets its samples)."""
        import pynvml as nv
        nv.nvmlInit()
        h = None
        if self.uuid:
            try:
                h = nv.nvmlDeviceGetHandleByUUID(self.uuid)
            except Exception:
                h = None
        if h is None:
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
        self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
        return nv, h

    def _run(self, nv, h):
        try:
            while True:
                mhz = nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)
                try:
                    reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
                except Exception:
                    reasons = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                try:
                    watts = nv.nvmlDeviceGetPowerUsage(h) / 1000.0
                except Exception:
                    watts = None
                self.samples.append((mhz, reasons, watts))
                if self._stop.wait(self.period):
                    break
        except Exception as e:
            self.samples.append(("error", str(e), None))

    def __enter__(self):
        try:
            nv, h = self._open()
        except Exception as e:  # NVML missing: report that instead of inventing clocks
            self.samples.append(("error", str(e), None))
            return self
        self._thread = threading.Thread(target=self._run, args=(nv, h), daemon=True)
        self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)

    def summary(self):
        good = [s for s in self.samples if s[0] != "error"]
        if not good:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["nvml_unavailable"], "samples": 0}
        names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
                 0x4: "sw_power_cap", 0x80: "hw_power_brake", 0x2: "applications_clocks_setting"}
        seen = set()
        for _, r, _ in good:
            for bit, n in names.items():
                if r & bit:
                    seen.add(n)
        watts = [w for _, _, w in good if w is not None]
        return {"sm_mhz": statistics.median(s[0] for s in good), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(seen), "samples": len(good), "power_w_max": max(watts) if watts else None}


def _dist():
    from paper_2607_10389_b200.replicas import rank_env
    return rank_env()


def oracle_step(sample_cur, sample_prev, chunk_bytes):
    """The CPU oracle's pass over one sample (same four calls as the GPU step)."""
    import numpy as np
    import oracle
    crc = oracle.checksum(sample_cur, chunk_bytes)
    dirty, _ = oracle.dirty_diff(sample_cur, sample_prev, chunk_bytes)
    wire, crc2, res = oracle.encode(sample_cur, chunk_bytes)
    out, _, r = oracle.decode_verify(wire, sample_cur.size, chunk_bytes)
    assert res.status == 0 and r.status == 0 and np.array_equal(out, sample_cur) and np.array_equal(crc, crc2)
    return int(dirty.sum())


def cpu_baseline(cur_host, prev_host, chunk_bytes, target_s=20.0):
    """Time the oracle, as it stands, on a bounded sample of the workload: once on one core, then
    on every core the process may use (one independent slice of the sample per thread: chunks are
    independent, and the oracle's C code runs outside the interpreter lock)."""
    from concurrent.futures import ThreadPoolExecutor
    n_chunks = cur_host.size // chunk_bytes
    n0 = min(cur_host.size, 8 * chunk_bytes)
    t = time.perf_counter()
    oracle_step(cur_host[:n0], prev_host[:n0], chunk_bytes)
    dt0 = time.perf_counter() - t
    per_chunk = dt0 / max(1, n0 // chunk_bytes)
    # single core: about half of the time budget
    chunks1 = max(8, min(n_chunks, int(0.5 * target_s / max(per_chunk, 1e-6))))
    n1 = min(cur_host.size, chunks1 * chunk_bytes)
    t = time.perf_counter()
    oracle_step(cur_host[:n1], prev_host[:n1], chunk_bytes)
    dt1 = time.perf_counter() - t
    single = n1 / dt1 / 1e9
    # all cores: every thread takes its own run of chunks of the sample, sized for a few seconds
    try:
        cores = len(os.sched_getaffinity(0))
    except AttributeError:
        cores = os.cpu_count() or 1
    per_thread = max(4, min(n_chunks, 32, int(0.3 * target_s / max(per_chunk, 1e-6))))     # bounded: host memory

    def work(i):
        lo = (i * per_thread) % max(1, n_chunks - per_thread + 1)
        a, b = lo * chunk_bytes, (lo + per_thread) * chunk_bytes
        oracle_step(cur_host[a:b], prev_host[a:b], chunk_bytes)

    t = time.perf_counter()
    with ThreadPoolExecutor(max_workers=cores) as pool:
        list(pool.map(work, range(cores)))
    dtp = time.perf_counter() - t
    total = cores * per_thread * chunk_bytes
    # courtesy strong baseline for the checksum step alone: the CPU's own CRC32C instruction
    hw_gbs = None
    import oracle
    hw = oracle.hw_crc_library()
    if hw is not None:
        nh = min(cur_host.size, 256 * chunk_bytes)
        t = time.perf_counter()
        for o in range(0, nh, chunk_bytes):
            hw.hw_crc32c_u64(cur_host[o:o + chunk_bytes].ctypes.data, min(chunk_bytes, nh - o))
        hw_gbs = nh / (time.perf_counter() - t) / 1e9
    return {"value": total / dtp / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
            "single_core_gbs": single, "checksum_only_sse42_single_core_gbs": hw_gbs,
            "sample": f"{cores} threads, each one pass of checksum+diff+encode+decode_verify over {per_thread} chunks "
                      f"({per_thread * chunk_bytes} bytes) of the workload's first {n_chunks} chunks, {dtp:.1f} s; "
                      f"single core: {n1} bytes in {dt1:.1f} s"}


def make_workload(name, device):
    import torch
    from paper_2607_10389_b200 import inputs
    cfg = inputs.CONFIGS[name]
    cur = inputs.make_cache(cfg, device)
    if cfg.kind == "llm":
        # previous snapshot: the same window before the last 16 tokens were appended
        prev, mask = inputs.before_append(cur, cfg, 16)
        torch.cuda.synchronize()
        return cfg, cur, prev, int(mask.sum())
    # previous snapshot: the same cache before a generation step rewrote 75 % of its chunks
    nc = (cfg.nbytes + cfg.chunk_bytes - 1) // cfg.chunk_bytes
    mask = inputs.step_pattern(nc, 30, 0.75, seed=cfg.seed + 100)
    prev = cur.clone()
    inputs.apply_step(prev, cfg.chunk_bytes, mask, seed=cfg.seed + 200)
    torch.cuda.synchronize()
    return cfg, cur, prev, int(mask.sum())


def precopy_loop(wm, inputs, cfg, cur, prev, dst, wire_a, ws_a, dev, peak, steps=20):
    """The pre-copy step loop: per generation step three quarters of the chunks are rewritten
    (contiguous token-block pattern), then wm_dirty_diff -> wm_encode of the dirty chunks only ->
    wm_decode_verify into the destination's live copy.  The rewritten caches of all steps are
    generated beforehand (the engine's own writes are not the mover's time), a first pass learns
    the image lengths and checks every step, and the timed passes enqueue whole runs without a
    host synchronisation: on one stream (the path's own cost per step), and on two streams, where
    step k's install runs beside step k+1's diff and encode, with every block count the callers
    can give the two sides (WM_OPT_BLOCKS)."""
    import torch
    N, C = cfg.nbytes, cfg.chunk_bytes
    nc = wm.num_chunks(N, C)
    wires = [wire_a, torch.empty_like(wire_a)]
    ws_b = wm.new_workspace(N, C, dev)
    src, dstream = torch.cuda.Stream(), torch.cuda.Stream()
    masks = [inputs.step_pattern(nc, cfg.shape[0], 0.75, seed=1000 + k) for k in range(steps)]
    states = [cur]
    for k in range(steps):
        nxt = states[-1].clone()
        inputs.apply_step(nxt, C, masks[k], seed=5000 + k)
        states.append(nxt)
    crc0 = torch.zeros(nc, dtype=torch.int32, device=dev)
    crc_src, crc_dst = torch.zeros_like(crc0), torch.zeros_like(crc0)
    dirty = torch.zeros(nc, dtype=torch.uint8, device=dev)
    n_dirty = torch.zeros(1, dtype=torch.int32, device=dev)
    res_e = [wm.new_result(dev) for _ in range(steps)]
    res_d = [wm.new_result(dev) for _ in range(steps)]
    # level the two sides first (full move)
    wm.wm_encode(cur, C, None, crc0, wires[0], ws_a, res_e[0])
    r = wm.read_result(res_e[0])
    wm.wm_decode_verify(wires[0], r.wire_len, dst, C, crc_dst, ws_a, res_d[0])
    if not wm.read_result(res_d[0]).ok or not torch.equal(dst, cur):
        raise SystemExit("pre-copy loop: levelling move failed")

    def level():
        dst.copy_(states[0])
        crc_src.copy_(crc0)
        crc_dst.copy_(crc0)

    # first pass: step by step with the results read on the host
    level()
    lens = []
    for k in range(steps):
        wm.wm_dirty_diff(states[k + 1], states[k], C, dirty, None, n_dirty, ws_a)
        wm.wm_encode(states[k + 1], C, dirty, crc_src, wires[0], ws_a, res_e[k])
        rr = wm.read_result(res_e[k])
        if not rr.ok or rr.n_present != int(masks[k].sum()):
            raise SystemExit(f"pre-copy loop: encode failed at step {k}: {rr.status_name}")
        lens.append((rr.wire_len, rr.n_present))
        wm.wm_decode_verify(wires[0], rr.wire_len, dst, C, crc_dst, ws_b, res_d[k])
        if not wm.read_result(res_d[k]).ok or not torch.equal(dst, states[k + 1]):
            raise SystemExit(f"pre-copy loop: step {k} did not arrive")

    def run(two_streams, blocks_src, blocks_dst):
        level()
        torch.cuda.synchronize()
        s2 = dstream if two_streams else src
        opt_s, opt_d = wm.opt_blocks(blocks_src), wm.opt_blocks(blocks_dst)
        enc_done = [torch.cuda.Event() for _ in range(steps)]
        dec_done = [torch.cuda.Event() for _ in range(steps)]
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(src)
        s2.wait_event(t0)
        for k in range(steps):
            wire = wires[k % 2]
            if two_streams and k >= 2:
                src.wait_event(dec_done[k - 2])          # the image buffer is free again
            wm.wm_dirty_diff(states[k + 1], states[k], C, dirty, None, n_dirty, ws_a, stream=src)
            wm.wm_encode_opt(states[k + 1], C, dirty, crc_src, wire, ws_a, res_e[k], opt_s, stream=src)
            if two_streams:
                enc_done[k].record(src)
                s2.wait_event(enc_done[k])
            wm.wm_decode_verify_opt(wire, lens[k][0], dst, C, crc_dst, ws_b, res_d[k], opt_d, stream=s2)
            if two_streams:
                dec_done[k].record(s2)
        src.wait_stream(s2)
        t1.record(src)
        torch.cuda.synchronize()
        for k in range(steps):
            if not (wm.read_result(res_e[k]).ok and wm.read_result(res_d[k]).ok):
                raise SystemExit(f"pre-copy loop: step {k} failed in a timed run")
        if not torch.equal(dst, states[-1]) or not torch.equal(crc_dst, crc_src):
            raise SystemExit("pre-copy loop: destination differs from the source after the last step")
        return t0.elapsed_time(t1) / steps

    variants = {}
    for name, two, bs, bd in (("one_stream", False, 0, 0), ("two_streams", True, 0, 0), ("two_streams_74_74", True, 74, 74),
                              ("two_streams_100_48", True, 100, 48), ("two_streams_48_100", True, 48, 100)):
        run(two, bs, bd)
        variants[name] = min(run(two, bs, bd) for _ in range(3))

    # the three calls of a step alone, back to back, on the last step's data
    def timed(fn, reps=20):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    k = steps - 1
    level()
    dst.copy_(states[k])
    wm.wm_dirty_diff(states[k + 1], states[k], C, dirty, None, n_dirty, ws_a)
    calls = {"dirty_diff_ms": timed(lambda: wm.wm_dirty_diff(states[k + 1], states[k], C, dirty, None, n_dirty, ws_a)),
             "encode_dirty_only_ms": timed(lambda: wm.wm_encode(states[k + 1], C, dirty, crc_src, wires[0], ws_a, res_e[k]))}
    crc_dst.copy_(crc_src)
    calls["decode_verify_dirty_only_ms"] = timed(lambda: wm.wm_decode_verify(wires[0], lens[k][0], dst, C, crc_dst, ws_b, res_d[k]))
    if not wm.read_result(res_d[k]).ok:
        raise SystemExit("pre-copy loop: per-call timing: decode failed")
    dirty_bytes = [min(n * C, N) for _, n in lens]
    mean_dirty = sum(dirty_bytes) / steps
    mean_wire = sum(w for w, _ in lens) / steps
    del states
    one = variants["one_stream"]
    best = min(variants, key=variants.get)
    return {"steps": steps, "dirty_fraction": mean_dirty / N, "wire_bytes_per_step": mean_wire,
            "ms_per_step": one, "dirty_gbs": mean_dirty / (one * 1e-3) / 1e9,
            "frac_of_hbm_peak": (2 * N + 2 * (mean_dirty + mean_wire)) / (one * 1e-3) / 1e9 / peak,
            "ms_per_step_by_schedule": variants, "best_schedule": best, "calls": calls,
            "note": "ms_per_step = device time of diff + encode(dirty chunks only) + decode-verify-install per step, all on one "
                    "stream, no host synchronisation inside the run, the engine's rewrites generated beforehand; frac_of_hbm_peak "
                    "counts 2 N read by the diff plus dirty bytes and wire bytes once on each side; the two-stream schedules run "
                    "step k's install beside step k+1's diff and encode, a_b = at most a blocks (SMs) for the source's encode kernel "
                    "and b for the destination's decode kernel (WM_OPT_BLOCKS)"}


def append_loop(wm, inputs, cfg, cur, dst, wire, ws, dev, steps=8):
    """The append-only run of the text-model cache: the window fills from cfg.fill to 0.727 in
    `steps` appends, one of which appends nothing.  Per step wm_dirty_diff -> wm_encode of the dirty
    chunks (zero-tile option) -> wm_decode_verify into the destination, on one stream, timed on
    the device; the caches of all steps are generated beforehand."""
    import torch
    N, C = cfg.nbytes, cfg.chunk_bytes
    nc = wm.num_chunks(N, C)
    sched = inputs.append_schedule(cfg, steps)
    states, masks = [cur], []
    for k, (first, count) in enumerate(sched):
        nxt = states[-1].clone()
        masks.append(inputs.append_tokens(nxt, cfg, first, count, seed=7000 + k))
        states.append(nxt)
    crc_src = torch.zeros(nc, dtype=torch.int32, device=dev)
    crc_dst = torch.zeros(nc, dtype=torch.int32, device=dev)
    dirty = torch.zeros(nc, dtype=torch.uint8, device=dev)
    n_dirty = torch.zeros(1, dtype=torch.int32, device=dev)
    res_e, res_d = wm.new_result(dev), wm.new_result(dev)
    wm.wm_encode_opt(cur, C, None, crc_src, wire, ws, res_e, wm.OPT_ZERO_TILES)
    r = wm.read_result(res_e)
    wm.wm_decode_verify_opt(wire, r.wire_len, dst, C, crc_dst, ws, res_d, 0)
    if not (r.ok and wm.read_result(res_d).ok and torch.equal(dst, cur)):
        raise SystemExit("append loop: levelling move failed")
    out = []
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    for k in range(steps):
        a, b = states[k + 1], states[k]
        lens = None
        for rep in range(2):                   # first time: lengths and checks; second time: timed, no host read inside
            if rep == 1:
                dst.copy_(b)
                crc_src.copy_(crc_keep)
                crc_dst.copy_(crc_keep)
                torch.cuda.synchronize()
                ev[0].record()
            else:
                crc_keep = crc_src.clone()
            wm.wm_dirty_diff(a, b, C, dirty, None, n_dirty, ws)
            wm.wm_encode_opt(a, C, dirty, crc_src, wire, ws, res_e, wm.OPT_ZERO_TILES)
            if rep == 0:
                rr = wm.read_result(res_e)
                if not rr.ok or rr.n_present != int(masks[k].sum()):
                    raise SystemExit(f"append loop: step {k}: encode failed or wrong dirty count")
                lens = rr
            wm.wm_decode_verify_opt(wire, lens.wire_len, dst, C, crc_dst, ws, res_d, 0)
            if rep == 1:
                ev[1].record()
            torch.cuda.synchronize()
            if not wm.read_result(res_d).ok or not torch.equal(dst, a):
                raise SystemExit(f"append loop: step {k} did not arrive")
        out.append({"fill_after": (sched[k][0] + sched[k][1]) / cfg.shape[3], "appended_tokens": sched[k][1],
                    "dirty_fraction": lens.n_present / nc, "wire_bytes": lens.wire_len, "payload_bytes": lens.payload_bytes,
                    "ms": ev[0].elapsed_time(ev[1])})
    del states
    return {"steps": out, "note": "one stream, device time of diff + encode(dirty chunks, zero-tile option) + decode-verify-install "
                                  "per append; the step that appends nothing is all clean: its image is the metadata alone"}


def leaf_mode(wm, cfg, cur, wire, ws, dev, W, peak, reps=20):
    """wm_encode_leaves / wm_decode_verify_leaves on layers x {key, value} separate tensors."""
    import torch
    N, C = cfg.nbytes, cfg.chunk_bytes
    nc = wm.num_chunks(N, C)
    n_leaves = cfg.shape[0] * cfg.shape[1]
    lb = N // n_leaves
    if lb % 16384:
        return None
    src = [cur[i * lb:(i + 1) * lb].clone() for i in range(n_leaves)]
    dst = [torch.empty_like(x) for x in src]
    ts, td = wm.make_leaf_table(src, dev), wm.make_leaf_table(dst, dev)
    crc = torch.zeros(nc, dtype=torch.int32, device=dev)
    crc_d = torch.zeros(nc, dtype=torch.int32, device=dev)
    res_e, res_d = wm.new_result(dev), wm.new_result(dev)
    flat = torch.empty_like(cur)

    def enc():
        wm.wm_encode_leaves(ts, N, C, None, crc, wire, ws, res_e)

    def dec():
        wm.wm_decode_verify_leaves(wire, W, td, N, C, crc_d, ws, res_d)

    def flatten():
        torch.cat(src, out=flat)

    def rehydrate():
        for i, x in enumerate(dst):
            x.copy_(flat[i * lb:(i + 1) * lb])

    enc()
    dec()
    if not (wm.read_result(res_e).ok and wm.read_result(res_d).ok and all(torch.equal(a, b) for a, b in zip(src, dst))):
        raise SystemExit("leaf mode: round trip failed")
    out = {"leaves": n_leaves, "leaf_bytes": lb}
    for name, fn in (("encode_leaves", enc), ("decode_verify_leaves", dec), ("flatten_copy", flatten),
                     ("rehydrate_copy", rehydrate)):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        out[name + "_ms"] = a.elapsed_time(b) / reps
    out["encode_frac_of_hbm_peak"] = (N + W) / (out["encode_leaves_ms"] * 1e-3) / 1e9 / peak
    out["decode_frac_of_hbm_peak"] = (N + W) / (out["decode_verify_leaves_ms"] * 1e-3) / 1e9 / peak
    out["note"] = "flatten_copy / rehydrate_copy: what a flat-buffer move spends besides wm_encode / wm_decode_verify"
    return out


def leaf_mode_paper_table(wm, inputs_mod, cfg, cur, dev, peak, reps=20):
    """The leaf calls on a table shaped like the paper's movable set: 450 leaves (420 tensors of
    seeded random sizes and 30 flags of 2 to 64 bytes in between) adding up to 1,670,124,960 bytes,
    filled with the first bytes of the workload's cache.  Most tiles then begin off a 16-byte
    boundary inside their leaf and some cross leaves; beside it the flat calls on the same bytes."""
    import torch
    N, C = inputs_mod.PAPER_CACHE_BYTES, cfg.chunk_bytes
    if cur.numel() < N:
        return None
    sizes = inputs_mod.paper_leaf_sizes()
    nc = wm.num_chunks(N, C)
    src, o = [], 0
    for n in sizes:
        src.append(cur[o:o + n].clone())
        o += n
    dst = [torch.empty_like(x) for x in src]
    ts, td = wm.make_leaf_table(src, dev), wm.make_leaf_table(dst, dev)
    ws = wm.new_workspace(N, C, dev)
    wire = torch.empty(wm.wire_bound(N, C), dtype=torch.uint8, device=dev)
    wire_flat = torch.empty_like(wire)
    flat_dst = torch.empty(N, dtype=torch.uint8, device=dev)
    crc = torch.zeros(nc, dtype=torch.int32, device=dev)
    crc_d = torch.zeros(nc, dtype=torch.int32, device=dev)
    res_e, res_d = wm.new_result(dev), wm.new_result(dev)
    wm.wm_encode_leaves(ts, N, C, None, crc, wire, ws, res_e)
    r = wm.read_result(res_e)
    wm.wm_encode(cur[:N], C, None, crc_d, wire_flat, ws, res_d)
    rf = wm.read_result(res_d)
    if not (r.ok and rf.ok and r.wire_len == rf.wire_len and torch.equal(wire[: r.wire_len], wire_flat[: r.wire_len])):
        raise SystemExit("leaf mode (paper table): the image differs from the flat call's")
    W = r.wire_len
    wm.wm_decode_verify_leaves(wire, W, td, N, C, crc_d, ws, res_d)
    if not (wm.read_result(res_d).ok and all(torch.equal(a, b) for a, b in zip(src, dst))):
        raise SystemExit("leaf mode (paper table): round trip failed")
    calls = (("encode_leaves", lambda: wm.wm_encode_leaves(ts, N, C, None, crc, wire, ws, res_e)),
             ("decode_verify_leaves", lambda: wm.wm_decode_verify_leaves(wire, W, td, N, C, crc_d, ws, res_d)),
             ("encode_flat", lambda: wm.wm_encode(cur[:N], C, None, crc, wire_flat, ws, res_e)),
             ("decode_verify_flat", lambda: wm.wm_decode_verify(wire_flat, W, flat_dst, C, crc_d, ws, res_d)))
    edges, o = [], 0
    for n in sizes[:-1]:
        o += n
        edges.append(o)
    out = {"leaves": len(sizes), "nbytes": N, "wire_bytes": W,
           "tiles_that_cross_leaves": len({e // 16384 for e in edges if e % 16384}),
           "leaf_starts_off_16_bytes": sum(1 for e in edges if e % 16)}
    for name, fn in calls:
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        out[name + "_ms"] = a.elapsed_time(b) / reps
    out["encode_frac_of_hbm_peak"] = (N + W) / (out["encode_leaves_ms"] * 1e-3) / 1e9 / peak
    out["decode_frac_of_hbm_peak"] = (N + W) / (out["decode_verify_leaves_ms"] * 1e-3) / 1e9 / peak
    return out


def tail_schedule(wm, cfg, cur, shadow, wire, ws, dev, W, reps=8, super_mbs=(64, 128, 256)):
    """Verification placement: the move cut into super-chunks on three streams (encode, a device-to-device
    copy standing in for the wire, decode + verify), against the same three stages run one after the
    other on the whole cache.  `exposed_ms` is what remains after the last wire byte has arrived."""
    import statistics
    import torch
    from paper_2607_10389_b200 import tail_schedule as ts
    N, C = cfg.nbytes, cfg.chunk_bytes
    nc = wm.num_chunks(N, C)
    crc_s = torch.zeros(nc, dtype=torch.int32, device=dev)
    crc_d = torch.zeros(nc, dtype=torch.int32, device=dev)
    res_e, res_d = wm.new_result(dev), wm.new_result(dev)
    recv = torch.empty(W, dtype=torch.uint8, device=dev)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    tot, exp = [], []
    for i in range(reps + 2):
        torch.cuda.synchronize()
        ev[0].record()
        wm.wm_encode(cur, C, None, crc_s, wire, ws, res_e)
        wl = wm.read_result(res_e).wire_len              # the sender learns the image length
        recv[:wl].copy_(wire[:wl], non_blocking=True)
        ev[1].record()
        wm.wm_decode_verify(recv, wl, shadow, C, crc_d, ws, res_d)
        ev[2].record()
        torch.cuda.synchronize()
        if i >= 2:
            tot.append(ev[0].elapsed_time(ev[2]))
            exp.append(ev[1].elapsed_time(ev[2]))
    if not wm.read_result(res_d).ok:
        raise SystemExit("tail schedule: sequential move failed")
    out = {"sequential": {"total_ms": statistics.median(tot), "exposed_ms": statistics.median(exp)}, "pipelined": []}
    for mb in super_mbs:
        sup = mb << 20
        if sup % C or sup >= N:
            continue
        sched = ts.TailSchedule(N, C, sup, dev)
        tot, exp = [], []
        for i in range(reps + 2):
            shadow[:4096].zero_()
            rep = sched.move(cur, shadow, crc_s, crc_d)
            if not rep.ok:
                raise SystemExit("tail schedule: a part failed")
            if i >= 2:
                tot.append(rep.total_ms)
                exp.append(rep.exposed_ms)
        if not torch.equal(shadow, cur):
            raise SystemExit("tail schedule: destination differs from the source")
        out["pipelined"].append({"super_mib": mb, "parts": len(sched.parts), "total_ms": statistics.median(tot),
                                 "exposed_ms": statistics.median(exp), "launches": sched.launches})
        del sched
    out["note"] = ("total = first encode starts -> last verification ends; exposed = last wire copy ends -> last "
                   "verification ends; the wire is a device-to-device copy; medians of %d moves" % reps)
    return out


def entropy_option(wm, cfg, cur, shadow, wire, ws, dev, W_plain, peak, reps=20):
    """The ENT option (entropy-coded exponents): ratio and call times beside the default format's."""
    import torch
    N, C = cfg.nbytes, cfg.chunk_bytes
    nc = wm.num_chunks(N, C)
    crc = torch.zeros(nc, dtype=torch.int32, device=dev)
    crc_d = torch.zeros(nc, dtype=torch.int32, device=dev)
    res_e, res_d = wm.new_result(dev), wm.new_result(dev)
    wm.entropy_enable(True)
    try:
        wm.wm_encode(cur, C, None, crc, wire, ws, res_e)
        r = wm.read_result(res_e)
        if not r.ok:
            raise SystemExit("entropy option: encode failed")
        W = r.wire_len
        wm.wm_decode_verify(wire, W, shadow, C, crc_d, ws, res_d)
        if not (wm.read_result(res_d).ok and torch.equal(shadow, cur) and torch.equal(crc, crc_d)):
            raise SystemExit("entropy option: round trip failed")
        out = {"wire_bytes": W, "ratio": W / N, "ratio_default_format": W_plain / N}
        for name, fn in (("encode", lambda: wm.wm_encode(cur, C, None, crc, wire, ws, res_e)),
                         ("decode_verify", lambda: wm.wm_decode_verify(wire, W, shadow, C, crc_d, ws, res_d))):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(reps):
                fn()
            b.record()
            torch.cuda.synchronize()
            ms = a.elapsed_time(b) / reps
            out[name + "_ms"] = ms
            out[name + "_raw_gbs"] = N / (ms * 1e-3) / 1e9
            out[name + "_frac_of_hbm_peak"] = (N + W) / (ms * 1e-3) / 1e9 / peak
    finally:
        wm.entropy_enable(False)
    out["note"] = ("wm_entropy_enable(1): fixed prefix code of the exponents, a share's strands one behind the other with "
                   "their lengths written down; whole calls back to back; bound by integer instruction issue (one "
                   "table look-up per codeword and lane)")
    return out


def run_reference(args):
    """Reference arm: the CPU oracle timed on the host cores, a bounded sample per step."""
    rank, _, world = _dist()
    if rank != 0:
        return
    import numpy as np
    from paper_2607_10389_b200 import inputs
    name = args.workload
    cfg = inputs.CONFIGS[name]
    sample_chunks = 16
    n = min(cfg.nbytes, sample_chunks * cfg.chunk_bytes)
    # the sample is the head of the workload's own cache: its first layers, drawn with the same
    # generator on the same kind of device as the GPU arm draws them (torch is plumbing here: it
    # makes the input, the timed work is the oracle's on the host cores)
    import torch
    draw_on = "cuda" if torch.cuda.is_available() else "cpu"
    cur = inputs.make_cache(cfg, draw_on, head_bytes=n).cpu().numpy()[:n].copy()
    prev = cur.copy()
    nc = n // cfg.chunk_bytes
    mask = inputs.step_pattern(nc, 1, 0.75, seed=cfg.seed + 100).numpy()
    rng = np.random.default_rng(cfg.seed)
    for c in np.nonzero(mask)[0]:
        prev[c * cfg.chunk_bytes:(c + 1) * cfg.chunk_bytes] = rng.integers(0, 256, cfg.chunk_bytes, dtype=np.uint8)
    for _ in range(args.warmup):
        oracle_step(cur, prev, cfg.chunk_bytes)
    t = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(cur, prev, cfg.chunk_bytes)
    dt = (time.perf_counter() - t) / args.steps
    v = n / dt / 1e9
    sample = f"the first {n} bytes ({nc} chunks of {cfg.chunk_bytes}) of the {name} cache per step, single thread"
    print(json.dumps({
        "impl": "reference", "metric": METRIC,
        "value": v, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u8", "data": "synthetic",
        "config": {"workload": name, "nbytes": cfg.nbytes, "chunk_bytes": cfg.chunk_bytes, "sample_bytes": n},
        "cpu_baseline": {"value": v, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default="engine")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-loop", action="store_true", help="skip the pre-copy step loop")
    ap.add_argument("--zero-tiles", action="store_true", help="encoder option: all-zero tiles as table entries")
    ap.add_argument("--entropy", action="store_true", help="codec option: entropy-coded exponents (ENT tiles) in every call")
    ap.add_argument("--variant", default="plain", choices=["plain", "masked", "leaves", "paper_leaves", "xxh64", "xxh64_64k"],
                    help="with --profile: which calls make up a step (for profiler captures of the other kernel variants)")
    ap.add_argument("--profile", action="store_true",
                    help="profiler capture mode: round-trip check, warm-up and timed steps only")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        return run_reference(args)
    args.steps = 100 if args.steps is None else args.steps
    args.warmup = 5 if args.warmup is None else max(args.warmup, 3)
    if args.profile:
        args.no_e2e = args.no_cpu_baseline = args.no_loop = True

    import numpy as np
    import torch
    from paper_2607_10389_b200 import binding as wm
    from paper_2607_10389_b200 import inputs as inputs_mod

    rank, local_rank, world = _dist()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    from paper_2607_10389_b200.replicas import Replicas
    group = Replicas("nccl", dev)
    barrier, max_over_ranks = group.barrier, group.max_over_ranks

    wm.zero_tiles_enable(args.zero_tiles)
    wm.entropy_enable(args.entropy)
    cfg, cur, prev, n_rewritten = make_workload(args.workload, dev)
    N, C = cfg.nbytes, cfg.chunk_bytes
    nc = wm.num_chunks(N, C)
    ws = wm.new_workspace(N, C, dev)
    cap = wm.wire_bound(N, C)
    wire = torch.empty(cap, dtype=torch.uint8, device=dev)
    shadow = torch.empty(N, dtype=torch.uint8, device=dev)
    crc_a = torch.zeros(nc, dtype=torch.int32, device=dev)
    crc_b = torch.zeros(nc, dtype=torch.int32, device=dev)
    crc_dst = torch.zeros(nc, dtype=torch.int32, device=dev)
    dirty = torch.zeros(nc, dtype=torch.uint8, device=dev)
    dirty_idx = torch.zeros(nc, dtype=torch.int32, device=dev)
    n_dirty = torch.zeros(1, dtype=torch.int32, device=dev)
    res_e, res_d = wm.new_result(dev), wm.new_result(dev)

    state = {"wire_len": cap}
    launches = {"n": 0}

    def call_checksum():
        wm.wm_checksum(cur, C, crc_a, ws)
        launches["n"] += wm.last_launch_count()

    def call_diff():
        wm.wm_dirty_diff(cur, prev, C, dirty, dirty_idx, n_dirty, ws)
        launches["n"] += wm.last_launch_count()

    def call_encode():
        wm.wm_encode(cur, C, None, crc_b, wire, ws, res_e)
        launches["n"] += wm.last_launch_count()

    def call_decode():
        wm.wm_decode_verify(wire, state["wire_len"], shadow, C, crc_dst, ws, res_d)
        launches["n"] += wm.last_launch_count()

    def step():
        call_checksum()
        call_diff()
        call_encode()
        call_decode()

    # first pass: learn wire_len, check the round trip before timing anything
    call_encode()
    r = wm.read_result(res_e)
    if not r.ok:
        raise SystemExit(f"encode failed: {r.status_name}")
    state["wire_len"] = r.wire_len
    step()
    rd = wm.read_result(res_d)
    if not rd.ok or not torch.equal(shadow, cur) or not torch.equal(crc_a, crc_b) or not torch.equal(crc_dst, crc_b):
        raise SystemExit(f"round trip failed: {rd.status_name}")
    if int(n_dirty.item()) != n_rewritten:
        raise SystemExit("dirty count differs from the generated pattern")
    W = r.wire_len

    if args.profile and args.variant != "plain":
        # profiler captures of the other kernel variants: a step is the calls that run them
        if args.variant == "masked":
            # a pre-copy round: diff against the previous snapshot, encode the dirty chunks only,
            # decode into a destination that holds the previous snapshot
            crc_prev = torch.zeros(nc, dtype=torch.int32, device=dev)
            wm.wm_checksum(prev, C, crc_prev, ws)
            wm.wm_dirty_diff(cur, prev, C, dirty, dirty_idx, n_dirty, ws)
            crc_m = crc_prev.clone()
            wm.wm_encode(cur, C, dirty, crc_m, wire, ws, res_e)
            wl = wm.read_result(res_e).wire_len

            def step():
                shadow.copy_(prev)
                crc_m.copy_(crc_prev)
                crc_dst.copy_(crc_prev)
                wm.wm_dirty_diff(cur, prev, C, dirty, dirty_idx, n_dirty, ws)
                wm.wm_encode(cur, C, dirty, crc_m, wire, ws, res_e)
                wm.wm_decode_verify(wire, wl, shadow, C, crc_dst, ws, res_d)
        elif args.variant in ("leaves", "paper_leaves"):
            if args.variant == "leaves":
                n_leaves = cfg.shape[0] * cfg.shape[1]
                sizes, n_l = [N // n_leaves] * n_leaves, N
            else:       # the paper-shaped table scaled to this cache: the same 450 sizes in proportion
                full = inputs_mod.paper_leaf_sizes()
                sizes = [max(2, s * N // inputs_mod.PAPER_CACHE_BYTES // 2 * 2) for s in full]
                sizes[-1] += N - sum(sizes)
                n_l = N
            src_l, o = [], 0
            for k in sizes:
                src_l.append(cur[o:o + k].clone())
                o += k
            dst_l = [torch.empty_like(x) for x in src_l]
            ts, td = wm.make_leaf_table(src_l, dev), wm.make_leaf_table(dst_l, dev)
            wm.wm_encode_leaves(ts, n_l, C, None, crc_b, wire, ws, res_e)
            wl = wm.read_result(res_e).wire_len

            def step():
                wm.wm_encode_leaves(ts, n_l, C, None, crc_b, wire, ws, res_e)
                wm.wm_decode_verify_leaves(wire, wl, td, n_l, C, crc_dst, ws, res_d)
        else:
            xc = C if args.variant == "xxh64" else 65536
            hashes = torch.zeros(wm.num_chunks(N, xc), dtype=torch.int64, device=dev)

            def step():
                wm.wm_checksum_xxh64(cur, xc, 0, hashes)
        step()
        torch.cuda.synchronize()
        if not (wm.read_result(res_e).ok and wm.read_result(res_d).ok):
            raise SystemExit("profile variant: a call failed")

    for _ in range(args.warmup):
        step()
    barrier()
    launches["n"] = 0
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    try:
        gpu_uuid = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_uuid = None
    # A cache that fits in L2 would be timed out of the cache after its first step: there a buffer
    # larger than L2 is written between the timed steps, each step in its own pair of events.
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev) if N <= L2_BYTES else None
    with ClockSampler(local_rank, gpu_uuid) as clk:
        if flush is None:
            ev0.record()
            for _ in range(args.steps):
                step()
            ev1.record()
            barrier()
            ms_total = max_over_ranks(ev0.elapsed_time(ev1))
        else:
            pairs = []
            for _ in range(args.steps):
                flush.zero_()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                step()
                b.record()
                pairs.append((a, b))
            barrier()
            ms_total = max_over_ranks(sum(a.elapsed_time(b) for a, b in pairs))
    ms_step = ms_total / args.steps
    gpu_launches = launches["n"]
    value = group.aggregate_gbs(N, ms_step)


    if args.profile:
        if rank == 0:
            print(json.dumps({"profile_mode": True, "workload": args.workload, "ms_per_step": ms_step,
                              "value": value, "gpu_launches": gpu_launches}))
        return

    # per-call and main-kernel times (separate pass; each call bracketed by events on the stream)
    wm.timing_enable(True)
    calls = {"checksum": (call_checksum, wm.KIND_CHECKSUM, N + 4 * nc),
             "dirty_diff": (call_diff, wm.KIND_DIFF, None),
             "encode": (call_encode, wm.KIND_ENCODE, N + W),
             "decode_verify": (call_decode, wm.KIND_DECODE, N + W)}
    reps = max(20, min(args.steps, 30))
    peak, peak_kind = _peaks()
    per_call = {}
    for name, (fn, kind, alg_bytes) in calls.items():
        # (1) calls enqueued back to back, one pair of events around all of them: the time a call
        #     takes on the device when the host keeps the stream fed (a call's first kernel is an
        #     ordinary launch, so consecutive calls do not overlap)
        wm.timing_enable(False)
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        cm = a.elapsed_time(b) / reps
        wm.timing_enable(True)
        # (2) one call at a time with a synchronize in between (adds the host's launch latency for
        #     the short kernels ahead of the main one) and the library's timer on the main kernel
        iso_ms, kern_ms = [], []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            iso_ms.append(a.elapsed_time(b))
            kern_ms.append(wm.timing_read_ms(kind))
        km = statistics.mean(kern_ms)
        entry = {"call_ms": cm, "call_ms_isolated": statistics.mean(iso_ms), "call_ms_isolated_min": min(iso_ms),
                 "kernel_ms": km, "kernel_ms_min": min(kern_ms), "raw_gbs": N / (cm * 1e-3) / 1e9, "reps": reps}
        if alg_bytes:
            entry["algorithmic_bytes"] = alg_bytes
            entry["kernel_traffic_gbs"] = alg_bytes / (km * 1e-3) / 1e9
            entry["frac_of_hbm_peak"] = entry["kernel_traffic_gbs"] / peak
            entry["call_frac_of_hbm_peak"] = alg_bytes / (cm * 1e-3) / 1e9 / peak
            entry["frac_of_nominal_8tbs"] = entry["kernel_traffic_gbs"] / 8000.0
        per_call[name] = entry
    wm.timing_enable(False)
    # verify-before-write decode (two passes over the image): back-to-back time per call
    for _ in range(3):
        wm.wm_decode_verify_strict(wire, state["wire_len"], shadow, C, crc_dst, ws, res_d)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        wm.wm_decode_verify_strict(wire, state["wire_len"], shadow, C, crc_dst, ws, res_d)
    b.record()
    torch.cuda.synchronize()
    if not wm.read_result(res_d).ok:
        raise SystemExit("strict decode failed")
    per_call["decode_verify_strict"] = {"call_ms": a.elapsed_time(b) / reps, "reps": reps,
                                        "note": "wm_decode_verify_strict: nothing is stored before the verdict"}
    # the checksum step with the CRC-32 polynomial of zlib (same kernels, other tables)
    crc_z = torch.zeros(nc, dtype=torch.int32, device=dev)
    for _ in range(3):
        wm.wm_checksum_poly(cur, C, wm.POLY_ZLIB, crc_z, ws)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        wm.wm_checksum_poly(cur, C, wm.POLY_ZLIB, crc_z, ws)
    b.record()
    torch.cuda.synchronize()
    zm = a.elapsed_time(b) / reps
    per_call["checksum_zlib_polynomial"] = {"call_ms": zm, "reps": reps,
                                            "call_frac_of_hbm_peak": (N + 4 * nc) / (zm * 1e-3) / 1e9 / peak}
    # XXH64 of every chunk (a serial chain per chunk: four threads of work each)
    h64 = torch.zeros(nc, dtype=torch.int64, device=dev)
    for _ in range(3):
        wm.wm_checksum_xxh64(cur, C, 0, h64)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        wm.wm_checksum_xxh64(cur, C, 0, h64)
    b.record()
    torch.cuda.synchronize()
    xm = a.elapsed_time(b) / reps
    per_call["checksum_xxh64"] = {"call_ms": xm, "reps": reps, "call_frac_of_hbm_peak": N / (xm * 1e-3) / 1e9 / peak,
                                  "note": "with 1 MiB chunks bound by the latency of XXH64's serial chain (four chains per "
                                          "chunk), not by memory; with 64 KiB chunks it runs at the memory rate"}
    # dirty diff: bytes it actually has to read (clean chunks in full on both sides)
    per_call["dirty_diff"]["note"] = f"{n_rewritten} of {nc} chunks dirty; clean chunks are read in full on both sides"

    enc = per_call["encode"]
    roofline = {"bound": "hbm", "kernel": "k_encode (fused checksum+encode)",
                "achieved": enc["kernel_traffic_gbs"], "peak": peak, "unit": "GB/s",
                "frac": enc["kernel_traffic_gbs"] / peak, "peak_source": f"of {peak_kind}",
                "traffic": NCU_TRAFFIC_BYTES.get(args.workload),
                "algorithmic_bytes_per_launch": N + W,
                "call_frac": enc["call_frac_of_hbm_peak"],
                "decode_frac": per_call["decode_verify"]["frac_of_hbm_peak"],
                "decode_call_frac": per_call["decode_verify"]["call_frac_of_hbm_peak"]}

    # pre-copy step loop (the fifth workload): per generation step the source rewrites three
    # quarters of the chunks, then diff -> encode(dirty only) on one stream and
    # decode-verify-install on another (two wire buffers), 20 steps, device-timed as a whole
    loop = None
    if not args.no_loop and args.workload in ("engine", "engine_256m"):
        loop = precopy_loop(wm, inputs_mod, cfg, cur, prev, shadow, wire, ws, dev, peak)

    # the append-only run of the text-model cache (window fill 0.249 -> 0.727, with an all-clean step)
    append = None
    if not args.no_loop and cfg.kind == "llm":
        append = append_loop(wm, inputs_mod, cfg, cur, shadow, wire, ws, dev)

    # leaf mode: the same cache held as one key and one value tensor per layer, encoded and
    # decoded in place, beside the flatten and rehydrate copies that this makes unnecessary
    leaf = None
    if not args.no_loop and cfg.kind in ("kv", "llm"):
        leaf = leaf_mode(wm, cfg, cur, wire, ws, dev, W, peak)
        if leaf is not None and args.workload == "engine":
            leaf["paper_table"] = leaf_mode_paper_table(wm, inputs_mod, cfg, cur, dev, peak)

    # the entropy-coded exponent option beside the default format
    ent = None
    if not args.no_loop and cfg.kind == "kv" and not args.zero_tiles and not args.entropy:
        ent = entropy_option(wm, cfg, cur, shadow, wire, ws, dev, W, peak)

    # verification placement: super-chunks on three streams against the whole cache stage by stage
    tail = None
    if not args.no_loop and args.workload in ("engine", "engine_256m"):
        tail = tail_schedule(wm, cfg, cur, shadow, wire, ws, dev, W)

    # end to end: host cache in (pinned), verified wire image and result records out
    e2e = None
    if not args.no_e2e:
        host_cache = torch.empty(N, dtype=torch.uint8, pin_memory=True)
        host_cache.copy_(cur)
        host_wire = torch.empty(W, dtype=torch.uint8, pin_memory=True)
        host_res = torch.empty(80, dtype=torch.uint8, pin_memory=True)
        e_steps = max(4, min(args.steps, 24))
        # Two sets of device buffers and three streams: copy-in, the path, copy-out.  While step k
        # runs on one set, step k+1's cache is already coming in on the other and step k-1's wire
        # image and result records are going out.  Every step still pays its own host->device copy
        # of the whole cache and its own device->host copy of the image inside the timed region.
        cin, work, out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
        curs = [cur, torch.empty_like(cur)]
        wires = [wire, torch.empty_like(wire)]
        res_es = [res_e, wm.new_result(dev)]
        res_ds = [res_d, wm.new_result(dev)]
        host_wires = [host_wire, torch.empty(W, dtype=torch.uint8, pin_memory=True)]
        host_ress = [host_res, torch.empty(80, dtype=torch.uint8, pin_memory=True)]
        done_out = [None, None]            # the set's last image has left the device
        done_work = [None, None]           # the set's last pass over its cache has ended

        def e2e_step(i):
            b = i & 1
            with torch.cuda.stream(cin):
                if done_work[b] is not None:
                    cin.wait_event(done_work[b])
                curs[b].copy_(host_cache, non_blocking=True)
                arrived = torch.cuda.Event()
                arrived.record(cin)
            with torch.cuda.stream(work):
                work.wait_event(arrived)
                if done_out[b] is not None:
                    work.wait_event(done_out[b])
                wm.wm_checksum(curs[b], C, crc_a, ws, stream=work)
                wm.wm_dirty_diff(curs[b], prev, C, dirty, dirty_idx, n_dirty, ws, stream=work)
                wm.wm_encode(curs[b], C, None, crc_b, wires[b], ws, res_es[b], stream=work)
                wm.wm_decode_verify(wires[b], W, shadow, C, crc_dst, ws, res_ds[b], stream=work)
                done_work[b] = torch.cuda.Event()
                done_work[b].record(work)
            with torch.cuda.stream(out):
                out.wait_event(done_work[b])
                host_wires[b].copy_(wires[b][:W], non_blocking=True)
                host_ress[b][:40].copy_(res_es[b], non_blocking=True)
                host_ress[b][40:].copy_(res_ds[b], non_blocking=True)
                done_out[b] = torch.cuda.Event()
                done_out[b].record(out)

        torch.cuda.synchronize()
        e2e_step(0)
        e2e_step(1)
        barrier()
        done_out, done_work = [None, None], [None, None]
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record(cin)
        for i in range(e_steps):
            e2e_step(i)
        with torch.cuda.stream(out):
            out.wait_event(done_out[(e_steps - 1) & 1])
            out.wait_event(done_out[e_steps & 1])
            t1.record(out)
        barrier()
        ok = all(int.from_bytes(h[:4].numpy().tobytes(), "little", signed=True) == 0 and
                 int.from_bytes(h[40:44].numpy().tobytes(), "little", signed=True) == 0 for h in host_ress)
        if not ok or not torch.equal(host_wires[0], host_wires[1]):
            raise SystemExit("end-to-end pass: a step failed or the two buffer sets disagree")
        e_ms = max_over_ranks(t0.elapsed_time(t1)) / e_steps
        e2e = {"value": group.aggregate_gbs(N, e_ms), "unit": "GB/s", "h2d_bytes_per_step": N,
               "d2h_bytes_per_step": W + 80, "steps": e_steps, "ms_per_step": e_ms,
               "note": "two buffer sets, three streams: step k runs while step k+1's cache comes in and step k-1's image goes out"}

    # the same step captured once in a CUDA graph and replayed (the calls never allocate or
    # synchronise): what is left of the host's launch work, which matters for small caches
    graph_ms = None
    try:
        gs = torch.cuda.Stream()
        with torch.cuda.stream(gs):
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=gs):
                step()
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        ga, gb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ga.record()
        for _ in range(min(args.steps, 50)):
            graph.replay()
        gb.record()
        torch.cuda.synchronize()
        graph_ms = ga.elapsed_time(gb) / min(args.steps, 50)
        if not wm.read_result(res_d).ok:
            raise SystemExit("graph replay: decode failed")
        del graph
    except RuntimeError as e:      # capture is an extra: report why it was not measured
        graph_ms = None
        print("graph replay not measured:", e, file=sys.stderr)
    launches["n"] = gpu_launches

    base = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample_n = min(N, 1024 * C)
        base = cpu_baseline(cur[:sample_n].cpu().numpy(), prev[:sample_n].cpu().numpy(), C)

    if rank == 0:
        clocks = clk.summary()
        out = {
            "metric": METRIC,
            "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "ms_per_step_graph_replay": graph_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "u8", "data": "synthetic",
            "config": {"workload": args.workload, "nbytes": N, "chunk_bytes": C, "shape": list(cfg.shape),
                       "wire_bytes": W, "ratio": W / N, "dirty_chunks": n_rewritten, "n_chunks": nc,
                       "l2": "inputs larger than L2 (no flush needed)" if flush is None else
                             "cache fits in L2: a 256 MiB buffer is written between the timed steps (each step in its own event pair)", "parallelism": "replicas only",
                       "zero_tiles": bool(args.zero_tiles), "entropy": bool(args.entropy)},
            "calls": per_call, "roofline": roofline, "precopy_loop": loop, "append_loop": append, "leaf_mode": leaf, "entropy_option": ent, "tail_schedule": tail,
            "cpu_baseline": base, "e2e": e2e,
            "gpu_launches": gpu_launches, "clocks": clocks,
        }
        print(json.dumps(out))
    group.close()


if __name__ == "__main__":
    main()
