"""wm_encode_opt / wm_decode_verify_opt: the options per call give the images and verdicts that the
process-wide switches give, without touching those switches."""
import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu
TILE = 16384


def _cache(n, seed):
    rng = np.random.default_rng(seed)
    a = ((rng.normal(size=(n + 1) // 2)).astype(np.float32).view(np.uint32) >> 16).astype("<u2").view(np.uint8)[:n].copy()
    a[2 * TILE:3 * TILE] = 0
    return a


@pytest.mark.parametrize("options,kw", [(0, {}), (1, {"zero_tiles": True}), (2, {"entropy": True}),
                                        (3, {"entropy": True, "zero_tiles": True})])
def test_options_per_call_match_the_oracle(options, kw):
    import torch
    from paper_2607_10389_b200 import binding as wm
    n, chunk = 9 * TILE + 77, 2 * TILE
    a = _cache(n, 5)
    want, want_crc, want_res = oracle.encode(a, chunk, **kw)
    nc = wm.num_chunks(n, chunk)
    ws = wm.new_workspace(n, chunk)
    wire = torch.empty(wm.wire_bound(n, chunk), dtype=torch.uint8, device="cuda")
    crc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    res = wm.new_result()
    wm.wm_encode_opt(torch.from_numpy(a).cuda(), chunk, None, crc, wire, ws, res, options)
    r = wm.read_result(res)
    assert r.status == 0 and np.array_equal(wire[: r.wire_len].cpu().numpy(), want)
    for strict in (0, wm.OPT_STRICT):
        dst = torch.full((n,), 0x11, dtype=torch.uint8, device="cuda")
        dcrc = torch.zeros(nc, dtype=torch.int32, device="cuda")
        wm.wm_decode_verify_opt(wire, r.wire_len, dst, chunk, dcrc, ws, res, (options & wm.OPT_ENTROPY) | strict)
        assert wm.read_result(res).status == 0 and np.array_equal(dst.cpu().numpy(), a)
        assert np.array_equal(dcrc.cpu().numpy().view(np.uint32), want_crc)
    # the other kind of image is a format error, and the process-wide switches were never touched
    dst = torch.zeros(n, dtype=torch.uint8, device="cuda")
    wm.wm_decode_verify_opt(wire, r.wire_len, dst, chunk, dcrc, ws, res, (options & wm.OPT_ENTROPY) ^ wm.OPT_ENTROPY)
    assert wm.read_result(res).status_name == "ERR_FORMAT"
    wm.wm_encode(torch.from_numpy(a).cuda(), chunk, None, crc, wire, ws, res)
    r0 = wm.read_result(res)
    assert np.array_equal(wire[: r0.wire_len].cpu().numpy(), oracle.encode(a, chunk)[0])


def test_options_leaf_form_and_bad_arguments():
    import torch
    from paper_2607_10389_b200 import binding as wm
    n, chunk = 8 * TILE, 2 * TILE
    a = _cache(n, 6)
    want, want_crc, _ = oracle.encode(a, chunk, entropy=True)
    leaves = [torch.from_numpy(a[:6 * TILE].copy()).cuda(), torch.from_numpy(a[6 * TILE:].copy()).cuda()]
    nc = wm.num_chunks(n, chunk)
    ws = wm.new_workspace(n, chunk)
    wire = torch.empty(wm.wire_bound(n, chunk), dtype=torch.uint8, device="cuda")
    crc = torch.zeros(nc, dtype=torch.int32, device="cuda")
    res = wm.new_result()
    wm.wm_encode_opt(None, chunk, None, crc, wire, ws, res, wm.OPT_ENTROPY, leaf_table=wm.make_leaf_table(leaves), nbytes=n)
    r = wm.read_result(res)
    assert r.status == 0 and np.array_equal(wire[: r.wire_len].cpu().numpy(), want)
    out = [torch.zeros_like(x) for x in leaves]
    wm.wm_decode_verify_opt(wire, r.wire_len, None, chunk, crc, ws, res, wm.OPT_ENTROPY | wm.OPT_STRICT,
                            leaf_table=wm.make_leaf_table(out), nbytes=n)
    assert wm.read_result(res).status == 0 and all(torch.equal(x, y) for x, y in zip(leaves, out))
    with pytest.raises(wm.WmError, match="ERR_ARG"):
        wm.wm_encode_opt(leaves[0], chunk, None, crc, wire, ws, res, 8)                      # unknown option bit
    with pytest.raises(wm.WmError, match="ERR_ARG"):
        wm.wm_encode_opt(leaves[0], chunk, None, crc, wire, ws, res, wm.OPT_STRICT)          # decode-only option
    with pytest.raises(wm.WmError, match="ERR_ARG"):
        wm.wm_decode_verify_opt(wire, r.wire_len, leaves[0], chunk, crc, ws, res, 16)


def test_two_host_threads_with_different_options():
    """Two threads of one process, each with its own stream, geometry, workspace and options, issue
    calls at the same time; both get the oracle's images (the per-thread geometry caches and the
    per-call options keep them apart)."""
    import threading
    import torch
    from paper_2607_10389_b200 import binding as wm
    jobs = [(11 * TILE + 5, 2 * TILE, wm.OPT_ENTROPY, {"entropy": True}), (16 * TILE, 4 * TILE, 0, {})]
    errors = []

    def work(k):
        try:
            n, chunk, opt, kw = jobs[k]
            a = _cache(n, 40 + k)
            want, want_crc, _ = oracle.encode(a, chunk, **kw)
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                src = torch.from_numpy(a).cuda()
                nc = wm.num_chunks(n, chunk)
                ws = wm.new_workspace(n, chunk)
                wire = torch.empty(wm.wire_bound(n, chunk), dtype=torch.uint8, device="cuda")
                crc = torch.zeros(nc, dtype=torch.int32, device="cuda")
                res = wm.new_result()
                dst = torch.zeros(n, dtype=torch.uint8, device="cuda")
                for _ in range(40):
                    wm.wm_encode_opt(src, chunk, None, crc, wire, ws, res, opt, stream=stream)
                    wm.wm_decode_verify_opt(wire, want.size, dst, chunk, crc, ws, res, opt, stream=stream)
                stream.synchronize()
                r = wm.read_result(res)
                assert r.status == 0 and np.array_equal(wire[: want.size].cpu().numpy(), want)
                assert np.array_equal(dst.cpu().numpy(), a) and np.array_equal(crc.cpu().numpy().view(np.uint32), want_crc)
        except BaseException as e:      # noqa: BLE001 - reported by the main thread
            errors.append(repr(e))

    threads = [threading.Thread(target=work, args=(k,)) for k in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
