"""Parity at the benchmark's full sizes, in the launch configuration bench.py times:
sampled problems against the oracle, plus properties that hold for every problem."""
import numpy as np
import pytest
import torch

from oracle import curdkv_oracle as orc
from paper_2509_15038_b200 import binding as cur
from paper_2509_15038_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu
DEV = "cuda"


def run_path(w, three_calls=False):
    """The path as bench.py times it: one curdkv_compress call (three_calls: the separate calls)."""
    K, V, seqlens = synth.make_kv(w, DEV)
    G = synth.make_G(w.d, w.r, seed=0)
    Gd = torch.as_tensor(G, device=DEV)
    sl = None if seqlens is None else torch.as_tensor(seqlens, device=DEV)
    desc = cur.make_desc(K, V, w.r, q_heads=w.q_heads, seqlens=sl)
    ws = cur.alloc_workspace(desc, w.budget, w.adaptive)
    if three_calls:
        scores, sums = cur.curdkv_score(K, V, Gd, desc, ws)
        idx, cnt, off = cur.curdkv_select(scores, desc, w.budget, num_sink=w.num_sink, window=w.window,
                                          adaptive=w.adaptive, alpha=w.alpha, workspace=ws)
        Ko, Vo = cur.curdkv_compact(K, V, desc, idx, cnt, off, packed=w.adaptive, workspace=ws)
    else:
        scores, sums, idx, cnt, off, Ko, Vo = cur.curdkv_compress(
            K, V, Gd, desc, w.budget, ws, num_sink=w.num_sink, window=w.window, adaptive=w.adaptive,
            alpha=w.alpha)
    assert cur.curdkv_device_status(ws) == 0
    return K, V, G, seqlens, scores, sums, idx, cnt, off, Ko, Vo


def check_global_properties(w, K, V, seqlens, scores, idx, cnt, Ko, Vo):
    LB, H = w.folded_batch, w.kv_heads
    lens = torch.full((LB,), w.n_max, device=DEV) if seqlens is None else torch.as_tensor(seqlens, device=DEV)
    k_eff = torch.clamp(lens, max=w.budget)
    assert torch.equal(cnt, k_eff[:, None].expand(LB, H).to(torch.int32))
    tot = scores.sum(-1)
    assert torch.all((tot - 1).abs()[lens > 0] < 1e-3)
    t = torch.arange(w.budget, device=DEV)[None, None, :]
    valid = t < cnt[..., None]
    assert torch.all(idx[~valid] == -1)
    assert torch.all((idx >= 0)[valid]) and torch.all((idx < lens[:, None, None])[valid])
    inc = (idx[..., 1:] > idx[..., :-1]) | ~valid[..., 1:]
    assert torch.all(inc)
    # the last `window` tokens of every sequence are kept: they are the tail of each index row
    wnd = torch.clamp(lens, max=w.window)
    last = torch.gather(idx, 2, (cnt - 1).clamp(min=0)[..., None].long())[..., 0]
    assert torch.all((last == (lens - 1)[:, None])[lens > 0][:, :])
    first_w = torch.gather(idx, 2, (cnt - wnd[:, None]).clamp(min=0)[..., None].long())[..., 0]
    assert torch.all((first_w == (lens - wnd)[:, None])[lens > 0])
    # gathered rows equal the source rows at the selected indices (independent torch indexing)
    for lb in range(0, LB, max(1, LB // 16)):
        ii = idx[lb].clamp(min=0).long()
        want_k = torch.gather(K[lb], 1, ii[..., None].expand(-1, -1, w.d))
        want_v = torch.gather(V[lb], 1, ii[..., None].expand(-1, -1, w.d))
        m = valid[lb][..., None].expand_as(want_k)
        assert torch.equal(Ko[lb][m], want_k[m]) and torch.equal(Vo[lb][m], want_v[m])


def check_sampled_problems(w, K, V, G, seqlens, scores, idx, cnt, samples):
    worst = 0.0
    for lb, h in samples:
        n = w.n_max if seqlens is None else int(seqlens[lb])
        Ku = synth.to_u16(K[lb, h])[None, None]
        Vu = synth.to_u16(V[lb, h])[None, None]
        sl = None if seqlens is None else np.array([n], dtype=np.int32)
        rs, _ = orc.score(Ku, Vu, G, seqlens=sl)
        worst = max(worst, pu.assert_scores_close(scores[lb, h].cpu().numpy()[None, None], rs,
                                                  f"{w.name} lb={lb} h={h}"))
        ridx, rcnt = orc.select_fixed(rs, w.budget, w.num_sink, w.window, seqlens=sl)
        c = int(rcnt[0, 0])
        assert int(cnt[lb, h]) == c
        forced = pu.forced_tokens(n, c, w.num_sink, w.window)
        pu.assert_selection_within_band(idx[lb, h, :c].cpu().numpy(), ridx[0, 0, :c], rs[0, 0], n,
                                        forced, f"{w.name} lb={lb} h={h}")
        eidx, _ = orc.select_fixed(scores[lb, h].cpu().numpy().astype(np.float64)[None, None],
                                   w.budget, w.num_sink, w.window, seqlens=sl)
        np.testing.assert_array_equal(idx[lb, h].cpu().numpy(), eidx[0, 0])
    return worst


def test_cfg3_full_size_three_calls_equal_the_single_call():
    """At the headline size the single call (fused score + select kernel) and the three separate
    calls give the same bits; run twice to catch anything that depends on timing."""
    w = synth.CONFIGS["cfg3"]
    a = run_path(w, three_calls=True)
    want = [t.clone() for t in a[4:8]] + [a[9][::16].clone(), a[10][::16].clone()]
    del a
    torch.cuda.empty_cache()
    for _ in range(2):
        b = run_path(w)
        got = list(b[4:8]) + [b[9][::16], b[10][::16]]
        for name, x, y in zip(("scores", "head_sums", "idx", "head_counts", "K_out", "V_out"), got, want):
            assert torch.equal(x, y), name
        del b, got
        torch.cuda.empty_cache()


def test_cfg3_full_size():
    w = synth.CONFIGS["cfg3"]
    K, V, G, seqlens, scores, sums, idx, cnt, off, Ko, Vo = run_path(w)
    check_global_properties(w, K, V, seqlens, scores, idx, cnt, Ko, Vo)
    rng = np.random.default_rng(3)
    samples = [(int(rng.integers(w.folded_batch)), int(rng.integers(w.kv_heads))) for _ in range(6)]
    samples += [(0, 0), (w.folded_batch - 1, w.kv_heads - 1)]
    worst = check_sampled_problems(w, K, V, G, seqlens, scores, idx, cnt, samples)
    assert worst < 1e-4


@pytest.mark.parametrize("budget", [128, 512, 2048])
def test_cfg5_ragged_full_size(budget):
    w = synth.shrink(synth.CONFIGS["cfg5"], budget=budget)
    K, V, G, seqlens, scores, sums, idx, cnt, off, Ko, Vo = run_path(w)
    check_global_properties(w, K, V, seqlens, scores, idx, cnt, Ko, Vo)
    order = np.argsort(seqlens[: w.batch])
    picks = [int(order[0]), int(order[-1]), int(order[len(order) // 2])]      # shortest, longest, median
    samples = [(b + w.batch * (i * 7 % w.layers), (3 * i) % w.kv_heads) for i, b in enumerate(picks)]
    check_sampled_problems(w, K, V, G, seqlens, scores, idx, cnt, samples)


def test_cfg4_adaptive_full_size():
    w = synth.CONFIGS["cfg4"]
    K, V, G, seqlens, scores, sums, idx, cnt, off, Ko, Vo = run_path(w)
    LB, H = w.folded_batch, w.kv_heads
    assert torch.all(cnt.sum(-1) == H * w.budget)
    floor_rows = max(int(np.floor(w.alpha * w.budget)), w.window)
    assert int(cnt.min()) >= floor_rows
    offs = off.cpu().numpy()
    np.testing.assert_array_equal(offs[1:] - offs[:-1], cnt.cpu().numpy().reshape(-1))
    assert offs[0] == 0 and offs[-1] == LB * H * w.budget
    gi = idx.cpu().numpy()
    for lb in (0, 17, LB - 1):                      # whole (layer) groups against the oracle
        Ku, Vu = synth.to_u16(K[lb])[None], synth.to_u16(V[lb])[None]
        rs, _ = orc.score(Ku, Vu, G)
        pu.assert_scores_close(scores[lb].cpu().numpy()[None], rs, f"cfg4 lb={lb}")
        # the oracle's adaptive rule on the GPU's fp32 scores: bit-exact
        eidx, ecnt, eoff = orc.select_adaptive(scores[lb].cpu().numpy().astype(np.float64)[None],
                                               w.budget, w.num_sink, w.window, w.alpha)
        np.testing.assert_array_equal(cnt[lb].cpu().numpy(), ecnt[0])
        base = offs[lb * H]
        np.testing.assert_array_equal(gi[base: base + eoff[-1]], eidx)
        # against the oracle's own fp64 scores: every token on which the two selections differ
        # lies inside the tie band of a cut
        ridx, rcnt, roff = orc.select_adaptive(rs, w.budget, w.num_sink, w.window, w.alpha)
        pu.assert_adaptive_within_band(gi[base: base + eoff[-1]], eoff, ridx, roff, rs[0], 0, H, w.n_max,
                                       w.num_sink, w.window, f"cfg4 lb={lb}")
        # gathered rows of this group
        rows = torch.as_tensor(gi[base: base + eoff[-1]].astype(np.int64), device=DEV)
        heads = torch.repeat_interleave(torch.arange(H, device=DEV), torch.as_tensor(ecnt[0], device=DEV))
        assert torch.equal(Ko[base: base + eoff[-1]], K[lb][heads, rows])
        assert torch.equal(Vo[base: base + eoff[-1]], V[lb][heads, rows])
