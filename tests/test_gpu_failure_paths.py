"""Failure paths on the GPU that never fault it: a bounded device-side wait that runs out, and
counters that no call ever wrote.  Each case ends in a status bit the host reads; the context
stays usable and later calls give the same bits as before.  Needs a B200."""
import time

import numpy as np
import pytest
import torch

from paper_2509_15038_b200 import binding as cur
from paper_2509_15038_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_bounded_wait_runs_out_and_the_stream_stays_usable():
    """The wait routine of the pipelined kernels, on a barrier nothing completes, with a limit of
    2 ms: the status word gets CURDKV_DEV_TIMEOUT, curdkv_device_status returns CURDKV_ERR_TIMEOUT,
    and a normal scoring call on the same stream and workspace afterwards is bit-identical to one
    made before."""
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=1, n_max=2048)
    K, V, _ = synth.make_kv(w, DEV)
    G = torch.as_tensor(synth.make_G(w.d, w.r, seed=0), device=DEV)
    desc = cur.make_desc(K, V, w.r, q_heads=w.q_heads)
    ws = cur.alloc_workspace(desc)
    before_scores, before_sums = cur.curdkv_score(K, V, G, desc, ws)
    assert cur.curdkv_device_status(ws, with_code=True) == (0, 0)

    t0 = time.perf_counter()
    cur.curdkv_selftest_bounded_wait(2_000_000, ws)
    code, flags = cur.curdkv_device_status(ws, with_code=True)
    waited = time.perf_counter() - t0
    assert flags & cur.DEV_TIMEOUT
    assert code == 5 and "timed out" in cur.status_string(code)
    assert 0.002 <= waited < 1.0                            # the limit was honoured, and only the limit

    after_scores, after_sums = cur.curdkv_score(K, V, G, desc, ws)     # clears the status word
    assert cur.curdkv_device_status(ws, with_code=True) == (0, 0)
    assert torch.equal(after_scores, before_scores) and torch.equal(after_sums, before_sums)


def test_gather_wait_for_a_head_that_never_arrives_runs_out():
    """The gather that curdkv_compress starts beside the last selections waits per head for a ready
    flag.  With a flag that nothing sets, the wait ends at its limit with CURDKV_DEV_TIMEOUT, nothing
    else in the workspace is touched, and the next call on the stream works as before."""
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=1, n_max=2048)
    K, V, _ = synth.make_kv(w, DEV)
    G = torch.as_tensor(synth.make_G(w.d, w.r, seed=0), device=DEV)
    desc = cur.make_desc(K, V, w.r, q_heads=w.q_heads)
    ws = cur.alloc_workspace(desc, w.budget)
    before = [t.clone() for t in cur.curdkv_compress(K, V, G, desc, w.budget, ws, window=w.window)]
    ws[512:] = 0x5a
    t0 = time.perf_counter()
    cur.curdkv_selftest_gather_wait(2_000_000, ws)
    code, flags = cur.curdkv_device_status(ws, with_code=True)
    waited = time.perf_counter() - t0
    assert flags & cur.DEV_TIMEOUT and code == 5
    assert 0.002 <= waited < 1.0
    assert bool((ws[512:] == 0x5a).all())
    after = cur.curdkv_compress(K, V, G, desc, w.budget, ws, window=w.window)
    assert cur.curdkv_device_status(ws, with_code=True) == (0, 0)
    assert all(torch.equal(x, y) for x, y in zip(before, after))
    for bad in (0, 2_000_000_000):
        with pytest.raises(cur.CurdkvError) as e:
            cur.curdkv_selftest_gather_wait(bad, ws)
        assert e.value.code == 1


def test_bounded_wait_limit_is_validated_on_the_host():
    ws = torch.zeros((256,), dtype=torch.uint8, device=DEV)
    before = cur.launch_count()
    for bad in (0, 2_000_000_000):
        with pytest.raises(cur.CurdkvError) as e:
            cur.curdkv_selftest_bounded_wait(bad, ws)
        assert e.value.code == 1
    assert cur.launch_count() == before


def test_compact_cuts_counts_the_layout_cannot_hold():
    """Per-head counts above the index stride, or negative (a buffer no selection wrote): the gather
    copies what the layout holds, flags CURDKV_DEV_BAD_INDEX and leaves the neighbouring head's
    rows and the guard margins alone."""
    B, H, n, d, k = 1, 3, 64, 128, 4
    K = torch.randn((B, H, n, d), device=DEV).to(torch.bfloat16)
    V = torch.randn((B, H, n, d), device=DEV).to(torch.bfloat16)
    desc = cur.make_desc(K, V, 32)
    ws = cur.alloc_workspace(desc)
    ws.zero_()
    idx = torch.tensor([[[0, 5, 7, 63], [1, 2, 3, 4], [9, 8, 7, 6]]], dtype=torch.int32, device=DEV)
    cnt = torch.tensor([[1000, -3, 2]], dtype=torch.int32, device=DEV)
    pad = torch.full((B * H * k + 8, d), 7.0, dtype=torch.bfloat16, device=DEV)
    Ko, Vo = pad[4:-4].view(B, H, k, d), pad.clone()[4:-4].view(B, H, k, d)
    cur.curdkv_compact(K, V, desc, idx, cnt, K_out=Ko, V_out=Vo, workspace=ws)
    assert cur.curdkv_device_status(ws) & cur.DEV_BAD_INDEX
    assert torch.equal(Ko[0, 0], K[0, 0, idx[0, 0].long()])           # cut to the 4 rows that exist
    assert torch.all(Ko[0, 1] == 7.0)                                  # negative count: nothing
    assert torch.equal(Ko[0, 2, :2], K[0, 2, idx[0, 2, :2].long()]) and torch.all(Ko[0, 2, 2:] == 7.0)
    assert torch.all(pad[:4] == 7.0) and torch.all(pad[-4:] == 7.0)


def test_cache_append_with_counters_nobody_initialised():
    """count[b] outside [0, capacity]: the append is clamped and flagged instead of writing before
    or beyond the cache."""
    B, H, d, cap, t = 2, 2, 128, 16, 4
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=1, batch=B, n_max=t, kv_heads=H, q_heads=H)
    K, V, _ = synth.make_kv(w, DEV)
    G = torch.as_tensor(synth.make_G(d, 32, seed=0), device=DEV)
    cache = cur.DeviceCache(B, H, cap, d, DEV)
    cache.count.copy_(torch.tensor([-5, 1000], dtype=torch.int32))
    cache.K.fill_(3.0)
    ws = cur.cache_workspace(B, H, t, cap, 8, DEV)
    cur.curdkv_cache_append(cache, K, V, G, ws)
    flags = cur.curdkv_device_status(ws)
    assert flags & cur.DEV_BAD_INDEX
    cnt = cache.count.cpu().numpy()
    np.testing.assert_array_equal(cnt, [t, cap])                      # -5 -> 0 (+4 rows), 1000 -> full
    assert torch.equal(cache.K[0, :, :t], K[0])
    assert torch.all(cache.K[1] == 3.0) and torch.all(cache.K[0, :, t:] == 3.0)
