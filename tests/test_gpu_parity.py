"""Parity of the CUDA path (through the C ABI) with the fp64 oracle.  Needs a B200."""
import numpy as np
import pytest
import torch

from oracle import curdkv_oracle as orc
from paper_2509_15038_b200 import binding as cur
from paper_2509_15038_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu
DEV = "cuda"


def gpu_score(K, V, G, seqlens=None, q_heads=None, score_mode=0, use_projection=1):
    sl = None if seqlens is None else torch.as_tensor(seqlens, dtype=torch.int32, device=DEV)
    Gd = None if G is None else torch.as_tensor(G, dtype=torch.float32, device=DEV).contiguous()
    r = 1 if G is None else G.shape[-1]
    desc = cur.make_desc(K, V, r, q_heads=q_heads, seqlens=sl, score_mode=score_mode,
                         use_projection=use_projection)
    ws = cur.alloc_workspace(desc)
    scores, sums = cur.curdkv_score(K, V, Gd, desc, ws)
    return desc, ws, scores, sums, sl


class Guarded:
    """Output buffers cut out of larger allocations filled with a guard pattern; `check()` asserts
    that no byte of the margins before and after any of them was written (compute-sanitizer not being
    available, this and the comparison with the oracle are the evidence that stores stay in bounds)."""

    MARGIN = 4096          # bytes on either side; keeps the 16-byte alignment of the views
    PATTERN = 0xA5

    def __init__(self):
        self.raw = []

    def empty(self, shape, dtype):
        nbytes = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        buf = torch.full((nbytes + 2 * self.MARGIN,), self.PATTERN, dtype=torch.uint8, device=DEV)
        self.raw.append((buf, nbytes))
        return buf[self.MARGIN: self.MARGIN + nbytes].view(dtype).view(shape)

    def check(self, what=""):
        for i, (buf, nbytes) in enumerate(self.raw):
            assert torch.all(buf[: self.MARGIN] == self.PATTERN), f"{what}: write before output buffer {i}"
            assert torch.all(buf[self.MARGIN + nbytes:] == self.PATTERN), f"{what}: write past output buffer {i}"


def full_pipeline_check(K, V, G, budget, s, w, seqlens=None, what="", **kw):
    B, H, n_max, d = K.shape
    sl = None if seqlens is None else torch.as_tensor(seqlens, dtype=torch.int32, device=DEV)
    Gd = None if G is None else torch.as_tensor(G, dtype=torch.float32, device=DEV).contiguous()
    desc = cur.make_desc(K, V, 1 if G is None else G.shape[-1], seqlens=sl, **kw)
    ws = cur.alloc_workspace(desc)
    guard = Guarded()
    scores, sums = cur.curdkv_score(K, V, Gd, desc, ws, scores=guard.empty((B, H, n_max), torch.float32),
                                    head_sums=guard.empty((B, H), torch.float32))
    idx, cnt, _ = cur.curdkv_select(scores, desc, budget, num_sink=s, window=w, workspace=ws,
                                    idx=guard.empty((B, H, budget), torch.int32),
                                    head_counts=guard.empty((B, H), torch.int32),
                                    head_offsets=guard.empty((B * H + 1,), torch.int32))
    Ko, Vo = guard.empty((B, H, budget, d), torch.bfloat16), guard.empty((B, H, budget, d), torch.bfloat16)
    Ko.zero_()
    Vo.zero_()
    cur.curdkv_compact(K, V, desc, idx, cnt, K_out=Ko, V_out=Vo, workspace=ws)
    assert cur.curdkv_device_status(ws) == 0
    guard.check(what)

    Ku, Vu = synth.to_u16(K), synth.to_u16(V)
    rs, rS = orc.score(Ku, Vu, G if G is not None else np.zeros((K.shape[-1], 1), np.float32),
                       seqlens=seqlens, score_mode=kw.get("score_mode", 0),
                       use_projection=kw.get("use_projection", 1))
    worst = pu.assert_scores_close(scores.cpu().numpy(), rs, what + " scores")
    np.testing.assert_allclose(sums.cpu().numpy(), rS, rtol=1e-4)
    ridx, rcnt = orc.select_fixed(rs, budget, num_sink=s, window=w, seqlens=seqlens)
    gi, gc = idx.cpu().numpy(), cnt.cpu().numpy()
    np.testing.assert_array_equal(gc, rcnt)
    B, H, n_max, _ = K.shape
    diffs = 0
    for b in range(B):
        n = n_max if seqlens is None else int(min(max(seqlens[b], 0), n_max))
        for h in range(H):
            c = rcnt[b, h]
            forced = pu.forced_tokens(n, c, s, w)
            diffs += pu.assert_selection_within_band(gi[b, h, :c], ridx[b, h, :c], rs[b, h], n, forced,
                                                     f"{what} b={b} h={h}")
            assert np.all(gi[b, h, c:] == -1)
    # gathered bytes: exact copies of the rows the GPU selected
    Kg, Vg = orc.compact(Ku, Vu, gi, gc)
    np.testing.assert_array_equal(synth.to_u16(Ko), Kg)
    np.testing.assert_array_equal(synth.to_u16(Vo), Vg)
    # selection in the GPU's own precision: the oracle's rule on the fp32 scores is bit-exact
    eidx, ecnt = orc.select_fixed(scores.cpu().numpy().astype(np.float64), budget, num_sink=s,
                                  window=w, seqlens=seqlens)
    np.testing.assert_array_equal(gi, eidx)
    return worst, diffs


def test_cfg1_full():
    w = synth.CONFIGS["cfg1"]
    K, V, _ = synth.make_kv(w, DEV)
    G = synth.make_G(w.d, w.r, seed=0)
    worst, diffs = full_pipeline_check(K, V, G, w.budget, w.num_sink, w.window, what="cfg1")
    assert worst < 1e-3


def test_cfg2_two_layers():
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=2)
    K, V, _ = synth.make_kv(w, DEV)
    G = synth.make_G(w.d, w.r, seed=0)
    full_pipeline_check(K, V, G, w.budget, w.num_sink, w.window, q_heads=w.q_heads, what="cfg2x2")


def test_ragged_tail_and_sinks():
    """n_max not a multiple of the 128-row tile, ragged lengths incl. 0, paper mode s = 4."""
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=1, batch=5, n_max=1000)
    K, V, _ = synth.make_kv(w, DEV)
    G = synth.make_G(w.d, 32, seed=0)
    lens = np.array([1000, 777, 128, 0, 1], dtype=np.int32)
    for s, win, k in ((4, 0, 100), (4, 16, 100), (0, 32, 300), (4, 8, 10), (4, 8, 2000)):
        full_pipeline_check(K, V, G, k, s, win, seqlens=lens, what=f"ragged s={s} w={win} k={k}")


def test_ragged_batch_larger_than_one_kernel_slice():
    """More ragged sequences than one sketch launch keeps prefix sums for: the batch is cut into
    slices; lengths include 0 and non-multiples of the tile."""
    B, H, n, d = 8200, 1, 256, 128
    g = torch.Generator(device=DEV).manual_seed(11)
    K = torch.randn((B, H, n, d), generator=g, device=DEV).to(torch.bfloat16)
    V = torch.randn((B, H, n, d), generator=g, device=DEV).to(torch.bfloat16)
    lens = np.random.default_rng(5).integers(0, n + 1, size=B).astype(np.int32)
    lens[:4] = [0, 1, 129, 256]
    G = synth.make_G(d, 32, seed=0)
    desc, ws, scores, sums, sl = gpu_score(K, V, G, lens)
    assert cur.curdkv_device_status(ws) == 0
    rs, rS = orc.score(synth.to_u16(K), synth.to_u16(V), G, seqlens=lens)
    pu.assert_scores_close(scores.cpu().numpy(), rs, "sliced ragged batch")
    np.testing.assert_allclose(sums.cpu().numpy(), rS, rtol=1e-4)
    idx, cnt, _ = cur.curdkv_select(scores, desc, 40, num_sink=2, window=8, workspace=ws)
    eidx, ecnt = orc.select_fixed(scores.cpu().numpy().astype(np.float64), 40, num_sink=2, window=8,
                                  seqlens=lens)
    np.testing.assert_array_equal(cnt.cpu().numpy(), ecnt)
    np.testing.assert_array_equal(idx.cpu().numpy(), eidx)


def test_odd_row_count_misaligned_score_rows():
    """n_max = 1001: score rows of odd heads start off 16-byte boundaries (scalar paths of the
    normaliser and the selection), and the last tile holds a single row."""
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=1, batch=2, n_max=1001, kv_heads=3, q_heads=3)
    K, V, _ = synth.make_kv(w, DEV)
    G = synth.make_G(w.d, 32, seed=0)
    full_pipeline_check(K, V, G, 150, 4, 16, what="n_max=1001")
    full_pipeline_check(K, V, G, 150, 0, 8, seqlens=np.array([1001, 897], dtype=np.int32), what="n_max=1001 ragged")


def test_strided_token_major_layout():
    """K, V stored [B, n, H, d] (token-major) and viewed as [B, H, n, d]."""
    B, H, n, d = 2, 4, 640, 128
    g = torch.Generator(device=DEV).manual_seed(7)
    Kb = torch.randn((B, n, H, d), generator=g, device=DEV).to(torch.bfloat16)
    Vb = torch.randn((B, n, H, d), generator=g, device=DEV).to(torch.bfloat16)
    K, V = Kb.permute(0, 2, 1, 3), Vb.permute(0, 2, 1, 3)
    full_pipeline_check(K, V, synth.make_G(d, 32), 64, 0, 8, what="strided")


@pytest.mark.parametrize("r", [20, 32, 64, 1])
def test_sketch_dims(r):
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=1, n_max=1536, kv_heads=3, q_heads=3)
    K, V, _ = synth.make_kv(w, DEV)
    full_pipeline_check(K, V, synth.make_G(w.d, r, seed=r), 200, 4, 32, what=f"r={r}")


def test_per_head_G():
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=2, n_max=512, kv_heads=4, q_heads=4)
    K, V, _ = synth.make_kv(w, DEV)
    G = synth.make_G(w.d, 32, seed=3, heads=4)
    full_pipeline_check(K, V, G, 100, 0, 16, what="per-head G")


@pytest.mark.parametrize("mode,proj", [(1, 1), (2, 1), (0, 0), (1, 0), (2, 0)])
def test_ablation_modes(mode, proj):
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=1, n_max=900, kv_heads=2, q_heads=2)
    K, V, _ = synth.make_kv(w, DEV)
    G = synth.make_G(w.d, 32) if proj else None
    full_pipeline_check(K, V, G, 90, 4, 16, score_mode=mode, use_projection=proj,
                        what=f"mode={mode} proj={proj}")


def test_orthogonal_G_closed_form_on_gpu():
    """G = I (r = d... here the first 64 coordinates): scores are partial row norms."""
    w = synth.shrink(synth.CONFIGS["cfg1"], n_max=384, kv_heads=2, q_heads=2)
    K, V, _ = synth.make_kv(w, DEV)
    G = np.zeros((128, 64), dtype=np.float32)
    G[:64, :64] = np.eye(64)
    desc, ws, scores, sums, _ = gpu_score(K, V, G, score_mode=1)
    want = (synth.u16_to_f64(synth.to_u16(K))[..., :64] ** 2).sum(-1)
    want /= want.sum(-1, keepdims=True)
    pu.assert_scores_close(scores.cpu().numpy(), want, "selector G")


def _select_case(scores_np, budget, s, w, seqlens=None, head_budgets=None):
    B, H, n = scores_np.shape
    sc = torch.as_tensor(scores_np, dtype=torch.float32, device=DEV)
    dummy = torch.empty((B, H, n, 8), dtype=torch.bfloat16, device=DEV)
    sl = None if seqlens is None else torch.as_tensor(seqlens, dtype=torch.int32, device=DEV)
    desc = cur.make_desc(dummy, dummy, 1, seqlens=sl)
    hb = None if head_budgets is None else torch.as_tensor(head_budgets, dtype=torch.int32, device=DEV)
    idx, cnt, _ = cur.curdkv_select(sc, desc, budget, num_sink=s, window=w, head_budgets=hb)
    ridx, rcnt = orc.select_fixed(sc.cpu().numpy().astype(np.float64), budget, num_sink=s, window=w,
                                  seqlens=seqlens, head_budgets=head_budgets)
    np.testing.assert_array_equal(cnt.cpu().numpy(), rcnt)
    np.testing.assert_array_equal(idx.cpu().numpy(), ridx)


@pytest.mark.parametrize("n", [3000, 12000, 30000])      # CTAs of 256, 512 and 1024 threads
def test_select_short_candidate_lists(n):
    """The keys that share the cut's leading digit are ranked directly when there are at most 192
    of them and by two more histogram passes otherwise: list lengths around that limit, cuts at
    the first, an inner and the last key of the list, duplicates among them."""
    rng = np.random.default_rng(n)
    for L in (1, 2, 64, 191, 192, 193, 400):
        sc = np.empty((1, 2, n), dtype=np.float32)
        for h in range(2):
            high = n // 3
            row = np.concatenate([2.0 + rng.random(high),                    # above the list's digit
                                  1.0 + rng.integers(0, 20, size=L) / 256.0,  # the list: few distinct values
                                  0.1 + 0.4 * rng.random(n - high - L)]).astype(np.float32)
            sc[0, h] = row[rng.permutation(n)]
        for j in sorted({1, (L + 1) // 2, L}):
            _select_case(sc, n // 3 + j, 0, 0)
            _select_case(sc, n // 3 + j + 6, 2, 4)


def test_select_edges_and_ties():
    rng = np.random.default_rng(0)
    sc = rng.random((2, 3, 5000)).astype(np.float32)
    for k, s, w in ((0, 0, 0), (1, 0, 0), (7, 4, 3), (6, 4, 3), (4999, 0, 0), (5000, 2, 2), (9000, 0, 0)):
        _select_case(sc, k, s, w)
    tied = (np.round(sc * 16) / 16).astype(np.float32)          # heavy ties incl. zeros
    for k in (10, 1000, 2500):
        _select_case(tied, k, 2, 5)
    _select_case(np.zeros((1, 2, 300), np.float32), 17, 0, 4)
    weird = sc.copy()
    weird[0, 0, ::7] = np.nan
    weird[0, 1, ::5] = -1.0
    weird[1, 2, 3] = np.inf
    _select_case(weird, 600, 1, 1)
    _select_case(sc, 800, 3, 9, seqlens=np.array([4097, 33], dtype=np.int32))
    _select_case(sc, 800, 0, 9, head_budgets=np.array([[800, 0, 13], [5000, 77, 1]], dtype=np.int32))
    tiny = rng.random((1, 1, 3)).astype(np.float32) * 1e-30      # tiny positive values keep their order
    _select_case(tiny, 2, 0, 0)


def test_select_long_rows():
    rng = np.random.default_rng(1)
    sc = (rng.random((1, 2, 131072)) ** 8).astype(np.float32)
    sc /= sc.sum(-1, keepdims=True)
    _select_case(sc, 6681, 0, 128)
    _select_case(sc, 6681, 4, 0)


def test_select_candidate_list_overflow_falls_back_to_sweeps():
    """Scores that share their leading 12 bits put more keys into the cut's digit than the
    shared-memory candidate list holds: fixed and adaptive selection must still be exact, ties included."""
    rng = np.random.default_rng(12)
    B, H, n = 2, 4, 20000
    near = (1.0 + rng.random((B, H, n)) * 2.0 ** -13).astype(np.float32)       # one leading digit for all
    _select_case(near, 3000, 4, 64)
    _select_case(near, 19000, 0, 0)
    coarse = (1.0 + np.floor(rng.random((B, H, n)) * 4) * 2.0 ** -20).astype(np.float32)   # four values: ties
    _select_case(coarse, 7000, 2, 10)
    _adaptive_case(near, 3000, 4, 64, 0.2)
    _adaptive_case(coarse, 7000, 2, 10, 0.5)
    mixed = near.copy()
    mixed[:, ::2] *= 3.0                                    # heads on different leading digits
    _adaptive_case(mixed, 5000, 0, 32, 0.1)
    long_rows = (1.0 + rng.random((1, 2, 60000)) * 2.0 ** -13).astype(np.float32)  # beyond the staged size
    _select_case(long_rows, 9000, 4, 128)


def test_compact_flags_bad_index_without_faulting():
    B, H, n, d = 1, 2, 64, 128
    K = torch.randn((B, H, n, d), device=DEV).to(torch.bfloat16)
    V = torch.randn((B, H, n, d), device=DEV).to(torch.bfloat16)
    desc = cur.make_desc(K, V, 32)
    ws = cur.alloc_workspace(desc)
    ws.zero_()
    idx = torch.tensor([[[0, 5, -1, 63], [1, 64, 2, 3]]], dtype=torch.int32, device=DEV)
    cnt = torch.full((B, H), 4, dtype=torch.int32, device=DEV)
    Ko, Vo = cur.curdkv_compact(K, V, desc, idx, cnt, workspace=ws)
    assert cur.curdkv_device_status(ws) & cur.DEV_BAD_INDEX
    assert torch.equal(Ko[0, 0, 1], K[0, 0, 5]) and torch.equal(Vo[0, 1, 3], V[0, 1, 3])
    assert torch.all(Ko[0, 0, 2] == 0) and torch.all(Vo[0, 1, 1] == 0)


def test_invalid_arguments_return_status_codes():
    K = torch.zeros((1, 2, 256, 128), dtype=torch.bfloat16, device=DEV)
    G = torch.zeros((128, 32), dtype=torch.float32, device=DEV)
    desc = cur.make_desc(K, K, 32)
    ws = cur.alloc_workspace(desc)
    before = cur.launch_count()
    with pytest.raises(cur.CurdkvError) as e:
        cur.curdkv_score(K, K, None, desc, ws)
    assert e.value.code == 1
    with pytest.raises(cur.CurdkvError) as e:
        cur.curdkv_score(K, K, G, desc, ws[:256])
    assert e.value.code == 3
    bad = cur.make_desc(K, K, 200)
    with pytest.raises(cur.CurdkvError) as e:
        cur.curdkv_score(K, K, G, bad, ws)
    assert e.value.code == 2
    scores = torch.zeros((1, 2, 256), device=DEV)
    with pytest.raises(cur.CurdkvError) as e:
        cur.curdkv_select(scores, desc, -1)
    assert e.value.code == 1
    with pytest.raises(cur.CurdkvError) as e:
        cur.curdkv_select(scores, desc, 8, adaptive=True, alpha=1.5)
    assert e.value.code == 1
    assert cur.launch_count() == before


def test_determinism_and_gqa_map():
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=2, n_max=4096)
    K, V, _ = synth.make_kv(w, DEV)
    G = synth.make_G(w.d, w.r)
    outs = []
    for _ in range(2):
        desc, ws, scores, sums, _ = gpu_score(K, V, G, q_heads=w.q_heads)
        idx, cnt, _ = cur.curdkv_select(scores, desc, 500, window=64)
        outs.append((scores.clone(), sums.clone(), idx.clone()))
    for a, b in zip(*outs):
        assert torch.equal(a, b)
    m = cur.curdkv_gqa_map(desc).cpu().tolist()
    assert m == [orc.kv_head_of_query(q, w.q_heads, w.kv_heads) for q in range(w.q_heads)]
    idx_q, cnt_q = cur.curdkv_gqa_expand(desc, idx, cnt)
    gi, gq = idx.cpu().numpy(), idx_q.cpu().numpy()
    for q in range(w.q_heads):
        h = orc.kv_head_of_query(q, w.q_heads, w.kv_heads)
        np.testing.assert_array_equal(gq[:, q], gi[:, h])
        np.testing.assert_array_equal(cnt_q.cpu().numpy()[:, q], cnt.cpu().numpy()[:, h])


# ---------------------------------------------------------------- AdaCurDKV

def _adaptive_case(scores_np, budget, s, w, alpha, seqlens=None):
    """GPU adaptive selection on given fp32 scores vs the oracle's rule on the same values."""
    B, H, n = scores_np.shape
    sc = torch.as_tensor(scores_np, dtype=torch.float32, device=DEV)
    dummy = torch.empty((B, H, n, 8), dtype=torch.bfloat16, device=DEV)
    sl = None if seqlens is None else torch.as_tensor(seqlens, dtype=torch.int32, device=DEV)
    desc = cur.make_desc(dummy, dummy, 1, seqlens=sl)
    idx, cnt, off = cur.curdkv_select(sc, desc, budget, num_sink=s, window=w, adaptive=True, alpha=alpha)
    ridx, rcnt, roff = orc.select_adaptive(sc.cpu().numpy().astype(np.float64), budget, s, w, alpha,
                                           seqlens=seqlens)
    np.testing.assert_array_equal(cnt.cpu().numpy(), rcnt)
    np.testing.assert_array_equal(off.cpu().numpy(), roff)
    np.testing.assert_array_equal(idx.cpu().numpy()[: roff[-1]], ridx)
    return idx, cnt, off


def test_adaptive_select_many_sequences_small_ctas():
    """More (layer, sequence) clusters than one round of 1024-thread CTAs holds: the kernel then runs
    with CTAs of 512 threads, two per SM, and lists of half the size.  Same rule, ties and ragged
    lengths included, and a row whose candidates overflow the shorter list."""
    rng = np.random.default_rng(77)
    B, H, n = 40, 8, 2500
    mass = rng.random((B, H, 1)) ** 3 + 0.01
    sc = (rng.random((B, H, n)) ** 4 * mass).astype(np.float32)
    _adaptive_case(sc, 300, 4, 16, 0.2)
    tied = (np.round(sc / sc.max() * 32) / 32).astype(np.float32)
    _adaptive_case(tied, 700, 2, 3, 0.5)
    lens = rng.integers(0, n + 1, size=B).astype(np.int32)
    lens[:3] = (n, 1, 0)
    _adaptive_case(sc, 500, 1, 7, 0.2, seqlens=lens)
    near = (1.0 + rng.random((B, H, 6000)) * 2.0 ** -13).astype(np.float32)   # one leading digit: list overflow
    _adaptive_case(near, 1000, 2, 10, 0.3)


@pytest.mark.parametrize("H", [1, 2, 3, 8, 16])
def test_adaptive_select_matches_oracle_rule(H):
    rng = np.random.default_rng(H)
    B, n = 3, 3000
    mass = rng.random((B, H, 1)) ** 3 + 0.01
    sc = (rng.random((B, H, n)) ** 4 * mass).astype(np.float32)
    for k, s, w, alpha in ((300, 0, 16, 0.2), (300, 4, 0, 0.0), (300, 4, 8, 1.0), (1, 0, 0, 0.5),
                           (40, 4, 40, 0.2), (2999, 0, 5, 0.2), (3000, 0, 0, 0.2), (5000, 2, 2, 0.3),
                           (0, 0, 0, 0.2)):
        _adaptive_case(sc, k, s, w, alpha)
    tied = (np.round(sc / sc.max() * 32) / 32).astype(np.float32)
    for k, alpha in ((100, 0.2), (1500, 0.5), (700, 0.0)):
        _adaptive_case(tied, k, 2, 3, alpha)
    _adaptive_case(sc, 500, 1, 7, 0.2, seqlens=np.array([3000, 41, 0], dtype=np.int32))
    one_head = np.zeros((1, H, n), dtype=np.float32)
    one_head[0, H // 2] = rng.random(n) + 1.0
    _adaptive_case(one_head, 200, 0, 10, 0.25)


def test_adaptive_select_long_rows_cfg4_shape():
    rng = np.random.default_rng(4)
    H, n = 8, 131072
    sc = (rng.random((1, H, n)) ** 6 * (rng.random((1, H, 1)) + 0.05)).astype(np.float32)
    sc /= sc.sum(-1, keepdims=True)
    w = synth.CONFIGS["cfg4"]
    _adaptive_case(sc, w.budget, w.num_sink, w.window, w.alpha)


def test_adaptive_pipeline_r64_packed_gather():
    """cfg4 recipe at n = 16384: r = 64 sketch, adaptive budgets, packed gather."""
    w = synth.shrink(synth.CONFIGS["cfg4"], layers=2, n_max=16384, budget=819 + 128)
    K, V, _ = synth.make_kv(w, DEV)
    G = synth.make_G(w.d, w.r, seed=0)
    desc, ws, scores, sums, _ = gpu_score(K, V, G, q_heads=w.q_heads)
    Ku, Vu = synth.to_u16(K), synth.to_u16(V)
    rs, rS = orc.score(Ku, Vu, G)
    pu.assert_scores_close(scores.cpu().numpy(), rs, "cfg4-shaped scores")
    P, cap = w.folded_batch * w.kv_heads, min(w.budget, w.n_max)
    guard = Guarded()
    idx, cnt, off = cur.curdkv_select(scores, desc, w.budget, num_sink=w.num_sink, window=w.window,
                                      adaptive=True, alpha=w.alpha, workspace=ws,
                                      idx=guard.empty((P * cap,), torch.int32),
                                      head_counts=guard.empty((w.folded_batch, w.kv_heads), torch.int32),
                                      head_offsets=guard.empty((P + 1,), torch.int32))
    Ko, Vo = cur.curdkv_compact(K, V, desc, idx, cnt, off, packed=True, workspace=ws,
                                K_out=guard.empty((P * cap, w.d), torch.bfloat16),
                                V_out=guard.empty((P * cap, w.d), torch.bfloat16))
    assert cur.curdkv_device_status(ws) == 0
    guard.check("packed adaptive outputs")
    gi, gc, go = idx.cpu().numpy(), cnt.cpu().numpy(), off.cpu().numpy()
    # the oracle's rule on the GPU's own fp32 scores: bit-exact
    eidx, ecnt, eoff = orc.select_adaptive(scores.cpu().numpy().astype(np.float64), w.budget,
                                           w.num_sink, w.window, w.alpha)
    np.testing.assert_array_equal(gc, ecnt)
    np.testing.assert_array_equal(go, eoff)
    np.testing.assert_array_equal(gi[: eoff[-1]], eidx)
    # against the oracle's fp64 scores: same totals, per-head budgets equal up to tokens whose
    # score lies within the tie band of a cut
    ridx, rcnt, roff = orc.select_adaptive(rs, w.budget, w.num_sink, w.window, w.alpha)
    assert np.all(gc.sum(-1) == rcnt.sum(-1)) and go[-1] == roff[-1]
    for b in range(w.folded_batch):
        pu.assert_adaptive_within_band(gi, go, ridx, roff, rs[b], b, w.kv_heads, w.n_max, w.num_sink,
                                       w.window, f"cfg4-shaped b={b}")
    # gathered bytes of the rows the GPU selected
    Kg, Vg = orc.compact(Ku, Vu, gi[: go[-1]], gc, go)
    np.testing.assert_array_equal(synth.to_u16(Ko)[: go[-1]], Kg)
    np.testing.assert_array_equal(synth.to_u16(Vo)[: go[-1]], Vg)


# ---------------------------------------------------------------- host-buffer entry point

@pytest.mark.parametrize("adaptive", [False, True])
def test_compress_host_matches_device_calls(adaptive):
    """curdkv_compress_host (pinned host buffers, chunked double-buffered pipeline) gives the
    same bits as the three device calls, with ragged lengths and a chunk size that does not
    divide the batch."""
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=1, batch=5, n_max=2048)
    K, V, _ = synth.make_kv(w, DEV)
    lens = np.array([2048, 1500, 0, 129, 2047], dtype=np.int32)
    G = synth.make_G(w.d, w.r)
    budget, s, win = 300, 2, 32
    desc, ws, scores, sums, sl = gpu_score(K, V, G, seqlens=lens)
    idx, cnt, off = cur.curdkv_select(scores, desc, budget, num_sink=s, window=win, adaptive=adaptive,
                                      alpha=0.2)
    Ko, Vo = cur.curdkv_compact(K, V, desc, idx, cnt, off, packed=adaptive)
    torch.cuda.synchronize()

    Kh, Vh = K.cpu().pin_memory(), V.cpu().pin_memory()
    hdesc = cur.make_desc(Kh, Vh, w.r)
    hdesc.seqlens = lens.ctypes.data
    bufs = cur.HostBuffers(hdesc, budget, adaptive, chunk_batch=2)
    for _ in range(2):      # the second call reuses the arena
        flags = cur.curdkv_compress_host(Kh, Vh, torch.as_tensor(G), hdesc, budget, bufs, num_sink=s,
                                         window=win, adaptive=adaptive, alpha=0.2)
        assert flags == 0
        np.testing.assert_array_equal(bufs.counts.numpy(), cnt.cpu().numpy())
        total = int(cnt.sum().item())
        if adaptive:
            np.testing.assert_array_equal(bufs.offsets.numpy(), off.cpu().numpy())
            np.testing.assert_array_equal(bufs.idx.numpy()[:total], idx.cpu().numpy()[:total])
            assert torch.equal(bufs.K_out[:total], Ko.cpu()[:total])
            assert torch.equal(bufs.V_out[:total], Vo.cpu()[:total])
        else:
            np.testing.assert_array_equal(bufs.idx.numpy(), idx.cpu().numpy())
            c = cnt.cpu().numpy()
            for b in range(5):
                for h in range(w.kv_heads):
                    assert torch.equal(bufs.K_out[b, h, : c[b, h]], Ko.cpu()[b, h, : c[b, h]])
                    assert torch.equal(bufs.V_out[b, h, : c[b, h]], Vo.cpu()[b, h, : c[b, h]])


def test_calls_can_be_captured_into_a_cuda_graph():
    """score -> select -> compact enqueue only kernels and memsets on the caller's stream, so the
    three calls can be captured once and replayed; the replay must reproduce the eager results."""
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=2, n_max=3000)
    K, V, _ = synth.make_kv(w, DEV)
    G = torch.as_tensor(synth.make_G(w.d, w.r, seed=0), device=DEV)
    desc = cur.make_desc(K, V, w.r, q_heads=w.q_heads)
    ws = cur.alloc_workspace(desc, 400, False)
    B, H = w.folded_batch, w.kv_heads
    scores = torch.empty((B, H, w.n_max), dtype=torch.float32, device=DEV)
    sums = torch.empty((B, H), dtype=torch.float32, device=DEV)
    idx = torch.empty((B, H, 400), dtype=torch.int32, device=DEV)
    Ko = torch.empty((B, H, 400, w.d), dtype=torch.bfloat16, device=DEV)
    Vo = torch.empty_like(Ko)
    cnt = torch.empty((B, H), dtype=torch.int32, device=DEV)
    off = torch.empty((B * H + 1,), dtype=torch.int32, device=DEV)

    def step():
        cur.curdkv_score(K, V, G, desc, ws, scores=scores, head_sums=sums)
        cur.curdkv_select(scores, desc, 400, num_sink=4, window=32, workspace=ws, idx=idx, head_counts=cnt,
                          head_offsets=off)
        cur.curdkv_compact(K, V, desc, idx, cnt, off, K_out=Ko, V_out=Vo, workspace=ws)

    step()
    torch.cuda.synchronize()
    want = [t.clone() for t in (scores, sums, idx, cnt, Ko, Vo)]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for t in (scores, sums, idx, cnt, Ko, Vo):
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert cur.curdkv_device_status(ws) == 0
    for a, b in zip(want, (scores, sums, idx, cnt, Ko, Vo)):
        assert torch.equal(a, b)
