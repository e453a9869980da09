"""curdkv_compress (one call; for the main shapes one kernel that scores, normalises and selects)
against the three separate calls, bit for bit, and through them against the oracle.  Needs a B200.

The single-kernel route is taken from one head per SM upwards (148 heads on a B200): the cases
below that are meant to reach it use 600 heads or more, the others cover the three-step route."""
import numpy as np
import pytest
import torch

from oracle import curdkv_oracle as orc
from paper_2509_15038_b200 import binding as cur
from paper_2509_15038_b200 import synth
from tests import parity_util as pu
from tests.test_gpu_parity import Guarded

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _both_ways(K, V, G, budget, s, w, seqlens=None, head_budgets=None, adaptive=False, alpha=0.2, what="",
               **desc_kw):
    """Runs the three calls and the single call on the same inputs and demands identical outputs."""
    B, H, n_max, d = K.shape
    sl = None if seqlens is None else torch.as_tensor(seqlens, dtype=torch.int32, device=DEV)
    hb = None if head_budgets is None else torch.as_tensor(head_budgets, dtype=torch.int32, device=DEV)
    Gd = None if G is None else torch.as_tensor(G, dtype=torch.float32, device=DEV).contiguous()
    desc = cur.make_desc(K, V, 1 if G is None else G.shape[-1], seqlens=sl, **desc_kw)
    ws = cur.alloc_workspace(desc, max(budget, 1), adaptive)
    scores, sums = cur.curdkv_score(K, V, Gd, desc, ws)
    idx, cnt, off = cur.curdkv_select(scores, desc, budget, num_sink=s, window=w, head_budgets=hb,
                                      adaptive=adaptive, alpha=alpha, workspace=ws)
    Ko, Vo = cur.curdkv_compact(K, V, desc, idx, cnt, off, packed=adaptive, workspace=ws)
    assert cur.curdkv_device_status(ws) == 0
    want = [t.clone() for t in (scores, sums, idx, cnt, Ko, Vo)]
    want_off = off.clone()

    guard = Guarded()
    P, cap = B * H, min(budget, n_max)
    rows = P * cap if adaptive else P * budget
    out = dict(scores=guard.empty((B, H, n_max), torch.float32), head_sums=guard.empty((B, H), torch.float32),
               idx=guard.empty((rows,), torch.int32) if adaptive else guard.empty((B, H, budget), torch.int32),
               head_counts=guard.empty((B, H), torch.int32), head_offsets=guard.empty((P + 1,), torch.int32),
               K_out=guard.empty((rows, d) if adaptive else (B, H, budget, d), torch.bfloat16),
               V_out=guard.empty((rows, d) if adaptive else (B, H, budget, d), torch.bfloat16))
    for rep in range(2):                                   # the second call reuses the workspace as the first left it
        out["K_out"].zero_()
        out["V_out"].zero_()
        out["scores"].fill_(-7.0)
        out["idx"].fill_(-9)
        cur.curdkv_compress(K, V, Gd, desc, budget, ws, num_sink=s, window=w, head_budgets=hb,
                            adaptive=adaptive, alpha=alpha, **out)
        assert cur.curdkv_device_status(ws) == 0
        guard.check(what)
        got = [out[k] for k in ("scores", "head_sums", "idx", "head_counts", "K_out", "V_out")]
        names = ("scores", "head_sums", "idx", "head_counts", "K_out", "V_out")
        total = int(want[3].sum())
        for name, g, t in zip(names, got, want):
            if adaptive and name in ("idx", "K_out", "V_out"):
                g, t = g[:total], t[:total]
            assert torch.equal(g.reshape(t.shape), t), f"{what}: {name} differs (call {rep})"
        if adaptive or budget > 0:
            assert torch.equal(out["head_offsets"], want_off), f"{what}: head_offsets differ"
    return desc, out


def test_compress_cfg1_and_cfg2_match_three_calls_and_oracle():
    for w in (synth.CONFIGS["cfg1"], synth.shrink(synth.CONFIGS["cfg2"], layers=2),
              synth.shrink(synth.CONFIGS["cfg2"], layers=76, n_max=1024, budget=204 + 64)):
        K, V, _ = synth.make_kv(w, DEV)
        G = synth.make_G(w.d, w.r, seed=0)
        _, out = _both_ways(K, V, G, w.budget, w.num_sink, w.window, q_heads=w.q_heads, what=w.name)
        # and directly against the oracle
        rs, rS = orc.score(synth.to_u16(K), synth.to_u16(V), G)
        pu.assert_scores_close(out["scores"].cpu().numpy(), rs, w.name)
        np.testing.assert_allclose(out["head_sums"].cpu().numpy(), rS, rtol=1e-4)
        ridx, rcnt = orc.select_fixed(rs, w.budget, w.num_sink, w.window)
        gi = out["idx"].cpu().numpy()
        for b in range(K.shape[0]):
            for h in range(K.shape[1]):
                c = int(rcnt[b, h])
                pu.assert_selection_within_band(gi[b, h, :c], ridx[b, h, :c], rs[b, h], w.n_max,
                                                pu.forced_tokens(w.n_max, c, w.num_sink, w.window), w.name)


def test_compress_ragged_lengths_zero_rows_and_odd_sizes():
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=1, batch=80, n_max=1000)
    K, V, _ = synth.make_kv(w, DEV)
    G = synth.make_G(w.d, 32, seed=0)
    lens = np.tile(np.array([1000, 777, 128, 0, 1], dtype=np.int32), 16)
    for s, win, k in ((4, 0, 100), (4, 16, 100), (0, 32, 300), (4, 8, 10), (4, 8, 2000), (0, 0, 1)):
        _both_ways(K, V, G, k, s, win, seqlens=lens, what=f"ragged s={s} w={win} k={k}")
    # n_max = 1001: score rows of odd heads are not 16-byte aligned, the last tile holds one row
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=1, batch=200, n_max=1001, kv_heads=3, q_heads=3)
    K, V, _ = synth.make_kv(w, DEV)
    _both_ways(K, V, G, 150, 4, 16, what="n_max=1001")
    _both_ways(K, V, G, 150, 0, 8, seqlens=np.tile(np.array([1001, 897], dtype=np.int32), 100),
               what="n_max=1001 ragged")


def test_compress_many_short_heads_and_long_rows():
    """More heads than a CTA's queue of finished heads holds at once, and rows longer than the
    standalone selection stages in shared memory."""
    g = torch.Generator(device=DEV).manual_seed(5)
    K = torch.randn((96, 8, 256, 128), generator=g, device=DEV).to(torch.bfloat16)
    V = torch.randn((96, 8, 256, 128), generator=g, device=DEV).to(torch.bfloat16)
    G = synth.make_G(128, 32, seed=2)
    _both_ways(K, V, G, 40, 2, 8, what="768 heads of 2 tiles")
    lens = np.random.default_rng(1).integers(0, 257, size=96).astype(np.int32)
    _both_ways(K, V, G, 40, 2, 8, seqlens=lens, what="768 ragged heads")
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=76, n_max=40000)
    K, V, _ = synth.make_kv(w, DEV)
    _both_ways(K, V, G, 4000, 4, 64, what="n=40000")


def test_compress_options_and_layouts():
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=200, n_max=1536, kv_heads=3, q_heads=3)
    K, V, _ = synth.make_kv(w, DEV)
    for r in (1, 20, 32):
        _both_ways(K, V, synth.make_G(w.d, r, seed=r), 200, 4, 32, what=f"r={r}")
    G = synth.make_G(w.d, 32, seed=0)
    _both_ways(K, V, G, 200, 4, 32, score_mode=1, what="key only")
    _both_ways(K, V, G, 200, 4, 32, score_mode=2, what="value only")
    _both_ways(K, V, G, 200, 4, 32, raw_scores=1, what="raw scores")
    _both_ways(K, V, G, 300, 0, 9, what="per-head budgets",
               head_budgets=np.tile(np.array([[300, 0, 13], [5000, 77, 1]], dtype=np.int32), (100, 1)))
    _both_ways(K, V, G, 0, 0, 0, what="budget 0")
    _both_ways(K, V, G, 2000, 4, 32, what="budget above the row count")      # keeps every row
    _both_ways(K, V, G, 40, 30, 30, what="forced rows beyond the budget")   # window first, then sinks
    _both_ways(torch.zeros_like(K), V, G, 100, 2, 4, what="all-zero keys")       # head sums of 0
    # token-major storage viewed as [B, H, n, d]
    g = torch.Generator(device=DEV).manual_seed(7)
    Kb = torch.randn((150, 640, 4, 128), generator=g, device=DEV).to(torch.bfloat16)
    Vb = torch.randn((150, 640, 4, 128), generator=g, device=DEV).to(torch.bfloat16)
    _both_ways(Kb.permute(0, 2, 1, 3), Vb.permute(0, 2, 1, 3), G, 64, 0, 8, what="strided")


def test_compress_shapes_that_take_the_three_step_route():
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=2, n_max=1024, kv_heads=4, q_heads=4)
    K, V, _ = synth.make_kv(w, DEV)
    G = synth.make_G(w.d, 32, seed=0)
    _both_ways(K, V, G, 120, 2, 16, adaptive=True, alpha=0.2, what="adaptive")
    _both_ways(K, V, synth.make_G(w.d, 64, seed=1), 120, 2, 16, what="r=64")
    _both_ways(K, V, synth.make_G(w.d, 32, seed=3, heads=4), 120, 0, 16, what="per-head G")
    _both_ways(K, V, None, 120, 4, 16, use_projection=0, what="no projection")
    _both_ways(K, V, G, 120, 4, 16, whiten=1, ridge=1e-4, what="whitened")
    _both_ways(K[:, :, :100], V[:, :, :100], G, 30, 2, 4, what="n_max < 128")


def test_compress_replays_from_a_cuda_graph():
    """The single call on a shape that takes the one-kernel route (a cooperative launch) can be captured
    once and replayed; the replay reproduces the eager results bit for bit."""
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=76, n_max=1024, budget=200)
    K, V, _ = synth.make_kv(w, DEV)
    G = torch.as_tensor(synth.make_G(w.d, w.r, seed=0), device=DEV)
    desc = cur.make_desc(K, V, w.r, q_heads=w.q_heads)
    ws = cur.alloc_workspace(desc, w.budget)
    out = cur.curdkv_compress(K, V, G, desc, w.budget, ws, num_sink=4, window=32)
    torch.cuda.synchronize()
    want = [t.clone() for t in out]
    names = ("scores", "head_sums", "idx", "head_counts", "head_offsets", "K_out", "V_out")
    bufs = dict(zip(names, out))

    def step():
        cur.curdkv_compress(K, V, G, desc, w.budget, ws, num_sink=4, window=32, **bufs)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for t in out:
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert cur.curdkv_device_status(ws) == 0
    for name, a, b in zip(names, want, out):
        assert torch.equal(a, b), name
