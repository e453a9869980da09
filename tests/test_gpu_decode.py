"""Generation-phase cache on the GPU (through the C ABI) against the step-by-step oracle and
against one application of Alg. 1 to the whole history.  Needs a B200."""
import numpy as np
import pytest
import torch

from oracle import curdkv_decode_oracle as dec
from oracle import curdkv_oracle as orc
from paper_2509_15038_b200 import binding as cur
from paper_2509_15038_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _history(B, H, N, d, seed):
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=1, batch=B, n_max=N, kv_heads=H, q_heads=H,
                     data_seed=seed)
    K, V, _ = synth.make_kv(w, DEV)
    return K, V


class _History:
    """fp64 scores l^K l^V (Alg. 1 (sketch, row norms, product)) of every real row a sequence has been fed, by position:
    what the tie-band rule measures a differing token against."""

    def __init__(self, B, H):
        self.raw = [[np.zeros((0,), np.float64) for _ in range(H)] for _ in range(B)]

    def add(self, Ku, Vu, G, t_new=None):
        raw = dec.raw_scores(Ku, Vu, G)
        for b, per_head in enumerate(self.raw):
            tb = raw.shape[2] if t_new is None else int(t_new[b])
            for h in range(len(per_head)):
                per_head[h] = np.concatenate([per_head[h], raw[b, h, :tb]])


def _assert_kept_within_band(got, want, hist_raw, s, w, what):
    """Kept positions of one head against the oracle's: equal outside the 1e-4 relative band around
    the oracle's cut (forced positions: below s, or among the last w of the history)."""
    total = len(hist_raw)
    forced = pu.forced_tokens(total, len(want), s, w)
    return pu.assert_selection_within_band(np.sort(got), want, hist_raw, total, forced, what)


def _run(K, V, G, schedule, k, s, w, capacity, t_new=None):
    """Feeds the history in chunks; compresses whenever a sequence could overflow and at the end."""
    B, H, N, d = K.shape
    Gd = torch.as_tensor(G, device=DEV)
    caches = [cur.DeviceCache(B, H, capacity, d, DEV), cur.DeviceCache(B, H, capacity, d, DEV)]
    ws = cur.cache_workspace(B, H, max(schedule), capacity, k, DEV)
    ref = dec.CacheOracle(B, H, d)
    Ku, Vu = synth.to_u16(K), synth.to_u16(V)
    hist = _History(B, H)
    live, at, held = 0, 0, 0
    for step, t in enumerate(schedule):
        if held + t > capacity:
            cur.curdkv_cache_compress(caches[live], caches[1 - live], k, ws, num_sink=s, window=w)
            ref.compress(k, s, w)
            live, held = 1 - live, min(held, k)
        tn = None if t_new is None else torch.as_tensor(t_new[step], dtype=torch.int32, device=DEV)
        cur.curdkv_cache_append(caches[live], K[:, :, at:at + t], V[:, :, at:at + t], Gd, ws, t_new=tn)
        ref.append(Ku[:, :, at:at + t], Vu[:, :, at:at + t], G, None if t_new is None else t_new[step])
        hist.add(Ku[:, :, at:at + t], Vu[:, :, at:at + t], G, None if t_new is None else t_new[step])
        at += t
        held += t
    cur.curdkv_cache_compress(caches[live], caches[1 - live], k, ws, num_sink=s, window=w)
    ref.compress(k, s, w)
    live = 1 - live
    assert cur.curdkv_device_status(ws) == 0
    return caches[live], ref, hist


def _compare(cache, ref, hist, k, s, w):
    B, H = ref.B, ref.H
    cnt = cache.count.cpu().numpy()
    np.testing.assert_array_equal(cache.total.cpu().numpy(), ref.total)
    pos, raw = cache.pos.cpu().numpy(), cache.raw.cpu().numpy()
    Ko, Vo = synth.to_u16(cache.K), synth.to_u16(cache.V)
    for b in range(B):
        for h in range(H):
            c = int(cnt[b])
            assert c == len(ref.pos[b][h])
            got = pos[b, h, :c]
            assert np.all(np.diff(got) > 0)
            want = ref.pos[b][h]
            # fp32 vs fp64 scores may only disagree inside the tie band of the cut
            _assert_kept_within_band(got, want, hist.raw[b][h], s, w, f"b={b} h={h}")
            both = np.intersect1d(got, want)
            gi = np.searchsorted(got, both)
            ri = np.searchsorted(want, both)
            np.testing.assert_array_equal(Ko[b, h][gi], ref.K[b][h][ri])
            np.testing.assert_array_equal(Vo[b, h][gi], ref.V[b][h][ri])
            np.testing.assert_allclose(raw[b, h][gi], ref.raw[b][h][ri], rtol=1e-3)


@pytest.mark.parametrize("k,s,w", [(64, 4, 0), (64, 0, 16), (100, 4, 8)])
def test_decode_chunks_match_oracle_and_one_shot(k, s, w):
    B, H, N, d, r = 3, 2, 700, 128, 32
    K, V = _history(B, H, N, d, seed=21)
    G = synth.make_G(d, r, seed=0)
    schedule = [256, 1, 1, 130, 7, 200, 64, 41]
    assert sum(schedule) == N
    cache, ref, hist = _run(K, V, G, schedule, k, s, w, capacity=k + 256)
    _compare(cache, ref, hist, k, s, w)
    # one application of Alg. 1 to the whole history keeps the same positions
    sc, _ = orc.score(synth.to_u16(K), synth.to_u16(V), G)
    idx, cnt = orc.select_fixed(sc, k, s, w)
    pos = cache.pos.cpu().numpy()
    for b in range(B):
        for h in range(H):
            forced = pu.forced_tokens(N, int(cnt[b, h]), s, w)
            pu.assert_selection_within_band(pos[b, h, :cnt[b, h]], idx[b, h, :cnt[b, h]], sc[b, h], N,
                                            forced, f"one-shot b={b} h={h}")


def test_decode_token_by_token_and_ragged_appends():
    B, H, N, d, r = 2, 2, 96, 128, 20
    K, V = _history(B, H, N, d, seed=22)
    G = synth.make_G(d, r, seed=1)
    cache, ref, hist = _run(K, V, G, [1] * N, 24, 4, 6, capacity=40)
    _compare(cache, ref, hist, 24, 4, 6)
    # sequences that bring different numbers of rows per step (the rest of the block is padding)
    schedule = [32, 32, 32]
    t_new = [np.array([32, 5], np.int32), np.array([0, 32], np.int32), np.array([17, 1], np.int32)]
    cache, ref, hist = _run(K, V, G, schedule, 24, 2, 4, capacity=64, t_new=t_new)
    _compare(cache, ref, hist, 24, 2, 4)


@pytest.mark.parametrize("k,s,w", [(64, 4, 0), (64, 0, 16), (100, 4, 8)])
def test_decode_in_place_keeps_the_same_rows(k, s, w):
    """In-place compression (rows stay put, survivors from the tail fill the holes): the cache ends
    up unordered but holds exactly the rows the ordered procedure and one-shot Alg. 1 keep."""
    B, H, N, d, r = 3, 2, 700, 128, 32
    K, V = _history(B, H, N, d, seed=31)
    G = synth.make_G(d, r, seed=0)
    Gd = torch.as_tensor(G, device=DEV)
    schedule = [256, 1, 1, 130, 7, 200, 64, 41]
    capacity = k + 256
    cache = cur.DeviceCache(B, H, capacity, d, DEV)
    ws = cur.cache_workspace(B, H, max(schedule), capacity, k, DEV)
    ref = dec.CacheOracle(B, H, d)
    Ku, Vu = synth.to_u16(K), synth.to_u16(V)
    hist = _History(B, H)
    hist.add(Ku, Vu, G)
    at = held = 0
    for t in schedule:
        if held + t > capacity:
            cur.curdkv_cache_compress_inplace(cache, k, ws, num_sink=s, window=w)
            ref.compress(k, s, w)
            held = min(held, k)
        cur.curdkv_cache_append(cache, K[:, :, at:at + t], V[:, :, at:at + t], Gd, ws)
        ref.append(Ku[:, :, at:at + t], Vu[:, :, at:at + t], G)
        at += t
        held += t
    cur.curdkv_cache_compress_inplace(cache, k, ws, num_sink=s, window=w)
    ref.compress(k, s, w)
    assert cur.curdkv_device_status(ws) == 0
    cnt = cache.count.cpu().numpy()
    pos, raw = cache.pos.cpu().numpy(), cache.raw.cpu().numpy()
    Ko, Vo = synth.to_u16(cache.K), synth.to_u16(cache.V)
    for b in range(B):
        for h in range(H):
            c = int(cnt[b])
            assert c == len(ref.pos[b][h])
            got = pos[b, h, :c]
            assert len(set(got.tolist())) == c                      # no slot twice
            # fp32 vs fp64 scores may only disagree inside the tie band of the cut
            _assert_kept_within_band(got, ref.pos[b][h], hist.raw[b][h], s, w, f"in place b={b} h={h}")
            for slot in range(c):                                   # every slot holds its token's rows
                np.testing.assert_array_equal(Ko[b, h, slot], Ku[b, h, got[slot]])
                np.testing.assert_array_equal(Vo[b, h, slot], Vu[b, h, got[slot]])
            order = np.argsort(got)
            both, gi, ri = np.intersect1d(got[order], ref.pos[b][h], return_indices=True)
            np.testing.assert_allclose(raw[b, h, :c][order][gi], ref.raw[b][h][ri], rtol=1e-3)


def _cache_state(cache):
    """Everything a cache holds, as host arrays cut to the rows in use."""
    cnt = cache.count.cpu().numpy()
    out = {"count": cnt, "total": cache.total.cpu().numpy()}
    for name in ("K", "V"):
        bits = synth.to_u16(getattr(cache, name))
        out[name] = [bits[b, :, : cnt[b]] for b in range(len(cnt))]
    for name in ("raw", "pos"):
        arr = getattr(cache, name).cpu().numpy()
        out[name] = [arr[b, :, : cnt[b]] for b in range(len(cnt))]
    return out


@pytest.mark.parametrize("k,s,w", [(64, 4, 0), (64, 0, 16), (100, 4, 8)])
def test_decode_step_call_equals_append_then_in_place_compression(k, s, w):
    """curdkv_cache_step (new rows copied and heads selected in one launch) leaves exactly the cache
    that curdkv_cache_append + curdkv_cache_compress_inplace leave, step after step, with full and
    with ragged blocks of new rows; and the kept rows are the oracle's, up to the tie band."""
    B, H, d, r, t = 3, 2, 128, 32, 48
    steps = 9
    K, V = _history(B, H, steps * t, d, seed=41)
    G = synth.make_G(d, r, seed=0)
    Gd = torch.as_tensor(G, device=DEV)
    rng = np.random.default_rng(k + s)
    t_news = [None] * 3 + [rng.integers(0, t + 1, size=B).astype(np.int32) for _ in range(steps - 3)]
    capacity = k + t
    one = cur.DeviceCache(B, H, capacity, d, DEV)
    two = cur.DeviceCache(B, H, capacity, d, DEV)
    ws1 = cur.cache_workspace(B, H, t, capacity, k, DEV)
    ws2 = cur.cache_workspace(B, H, t, capacity, k, DEV)
    ref = dec.CacheOracle(B, H, d)
    hist = _History(B, H)
    Ku, Vu = synth.to_u16(K), synth.to_u16(V)
    for i, tn in enumerate(t_news):
        Kb, Vb = K[:, :, i * t:(i + 1) * t], V[:, :, i * t:(i + 1) * t]
        tnd = None if tn is None else torch.as_tensor(tn, device=DEV)
        cur.curdkv_cache_step(one, Kb, Vb, Gd, k, ws1, num_sink=s, window=w, t_new=tnd)
        cur.curdkv_cache_append(two, Kb, Vb, Gd, ws2, t_new=tnd)
        cur.curdkv_cache_compress_inplace(two, k, ws2, num_sink=s, window=w)
        assert cur.curdkv_device_status(ws1) == 0 and cur.curdkv_device_status(ws2) == 0
        a, b_ = _cache_state(one), _cache_state(two)
        for name in ("count", "total"):
            np.testing.assert_array_equal(a[name], b_[name], err_msg=f"step {i}: {name}")
        for name in ("K", "V", "raw", "pos"):
            for x, y in zip(a[name], b_[name]):
                np.testing.assert_array_equal(x, y, err_msg=f"step {i}: {name}")
        ref.append(Ku[:, :, i * t:(i + 1) * t], Vu[:, :, i * t:(i + 1) * t], G, tn)
        hist.add(Ku[:, :, i * t:(i + 1) * t], Vu[:, :, i * t:(i + 1) * t], G, tn)
        ref.compress(k, s, w)
    st = _cache_state(one)
    for b in range(B):
        for h in range(H):
            got = st["pos"][b][h]
            assert len(got) == len(ref.pos[b][h])
            _assert_kept_within_band(got, ref.pos[b][h], hist.raw[b][h], s, w, f"step call b={b} h={h}")
            order = np.argsort(got)
            both, gi, ri = np.intersect1d(got[order], ref.pos[b][h], return_indices=True)
            np.testing.assert_array_equal(st["K"][b][h][order][gi], ref.K[b][h][ri])
            np.testing.assert_array_equal(st["V"][b][h][order][gi], ref.V[b][h][ri])
            np.testing.assert_allclose(st["raw"][b][h][order][gi], ref.raw[b][h][ri], rtol=1e-3)


def test_decode_step_call_with_a_cache_that_overflows_and_one_that_is_still_filling():
    """The step call on the edges: a cache still below its budget (every new row keeps its own slot),
    a block that does not fit under the capacity (the rows that fit are taken, the flag is raised),
    and a sequence that brings no rows.  Same cache and same flags as append + in-place compression."""
    B, H, d, r, t = 3, 2, 128, 32, 40
    K, V = _history(B, H, 4 * t, d, seed=47)
    Gd = torch.as_tensor(synth.make_G(d, r, seed=0), device=DEV)
    for k, capacity in ((100, 140), (60, 70)):              # filling for two steps / overflowing at once
        one = cur.DeviceCache(B, H, capacity, d, DEV)
        two = cur.DeviceCache(B, H, capacity, d, DEV)
        ws1 = cur.cache_workspace(B, H, t, capacity, k, DEV)
        ws2 = cur.cache_workspace(B, H, t, capacity, k, DEV)
        saw_full = False
        for i in range(4):
            Kb, Vb = K[:, :, i * t:(i + 1) * t], V[:, :, i * t:(i + 1) * t]
            tn = torch.as_tensor(np.array([t, 0, 17], dtype=np.int32), device=DEV) if i == 2 else None
            cur.curdkv_cache_step(one, Kb, Vb, Gd, k, ws1, num_sink=2, window=5, t_new=tn)
            cur.curdkv_cache_append(two, Kb, Vb, Gd, ws2, t_new=tn)
            f_append = cur.curdkv_device_status(ws2)
            cur.curdkv_cache_compress_inplace(two, k, ws2, num_sink=2, window=5)
            f1, f2 = cur.curdkv_device_status(ws1), f_append | cur.curdkv_device_status(ws2)
            assert f1 == f2, (k, i, f1, f2)
            saw_full |= bool(f1 & cur.DEV_CACHE_FULL)
            a, b_ = _cache_state(one), _cache_state(two)
            for name in ("count", "total"):
                np.testing.assert_array_equal(a[name], b_[name], err_msg=f"k={k} step {i}: {name}")
            for name in ("K", "V", "raw", "pos"):
                for x, y in zip(a[name], b_[name]):
                    np.testing.assert_array_equal(x, y, err_msg=f"k={k} step {i}: {name}")
        assert saw_full == (capacity == 70)                 # 40 held + 40 offered > 70; never above 140


def test_ordered_compression_of_a_cache_left_unordered():
    """append, in-place compression (which gives up the row order), append, then the ORDERED
    compression: sinks and window are found by position, so the result is the oracle's."""
    B, H, d, r = 2, 2, 128, 32
    k, s, w = 48, 4, 8
    K, V = _history(B, H, 200, d, seed=43)
    G = synth.make_G(d, r, seed=0)
    Gd = torch.as_tensor(G, device=DEV)
    Ku, Vu = synth.to_u16(K), synth.to_u16(V)
    capacity = 160
    a, b_ = cur.DeviceCache(B, H, capacity, d, DEV), cur.DeviceCache(B, H, capacity, d, DEV)
    ws = cur.cache_workspace(B, H, 100, capacity, k, DEV)
    ref = dec.CacheOracle(B, H, d)
    hist = _History(B, H)
    hist.add(Ku, Vu, G)
    cur.curdkv_cache_append(a, K[:, :, :100], V[:, :, :100], Gd, ws)
    ref.append(Ku[:, :, :100], Vu[:, :, :100], G)
    cur.curdkv_cache_compress_inplace(a, k, ws, num_sink=s, window=w)
    ref.compress(k, s, w)
    pos_now = a.pos.cpu().numpy()[:, :, :k]
    assert np.any(np.diff(pos_now, axis=-1) < 0), "the in-place form is expected to leave rows unordered"
    cur.curdkv_cache_append(a, K[:, :, 100:], V[:, :, 100:], Gd, ws)
    ref.append(Ku[:, :, 100:], Vu[:, :, 100:], G)
    cur.curdkv_cache_compress(a, b_, k, ws, num_sink=s, window=w)
    ref.compress(k, s, w)
    assert cur.curdkv_device_status(ws) == 0
    st = _cache_state(b_)
    np.testing.assert_array_equal(st["total"], ref.total)
    for b in range(B):
        for h in range(H):
            got = st["pos"][b][h]
            want = ref.pos[b][h]
            assert len(got) == len(want) == k
            assert set(range(s)) <= set(got.tolist()) and set(range(200 - w, 200)) <= set(got.tolist())
            _assert_kept_within_band(got, want, hist.raw[b][h], s, w, f"ordered after in place b={b} h={h}")
            for slot, token in enumerate(got):
                np.testing.assert_array_equal(st["K"][b][h][slot], Ku[b, h, token])
                np.testing.assert_array_equal(st["V"][b][h][slot], Vu[b, h, token])


def test_decode_overflow_is_flagged_not_written():
    B, H, d = 1, 1, 128
    K, V = _history(B, H, 64, d, seed=23)
    G = torch.as_tensor(synth.make_G(d, 32, seed=0), device=DEV)
    cache = cur.DeviceCache(B, H, 40, d, DEV)
    ws = cur.cache_workspace(B, H, 64, 40, 16, DEV)
    cur.curdkv_cache_append(cache, K, V, G, ws)
    flags = cur.curdkv_device_status(ws)
    assert flags & 0x4
    assert int(cache.count[0]) == 40 and int(cache.total[0]) == 64
    np.testing.assert_array_equal(synth.to_u16(cache.K)[0, 0], synth.to_u16(K)[0, 0, :40])
