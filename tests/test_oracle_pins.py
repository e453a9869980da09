"""Pins for the fp64 oracle: closed forms, statistics the Gaussian sketch must
obey, SVD leverage scores, invariants and brute force.  CPU only.

Each test is chosen so that one plausible mistake in the oracle (a dropped
term, a transposed G, a wrong index base, a wrong tie rule) makes it fail.
"""
import os

import numpy as np
import pytest

from oracle import curdkv_oracle as orc
from paper_2509_15038_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(x):
    return synth.f64_to_bf16_u16(np.asarray(x, dtype=np.float64))


def rand_kv(rng, B, H, n, d, scale=1.0):
    K = bf16_bits(rng.standard_normal((B, H, n, d)) * scale)
    V = bf16_bits(rng.standard_normal((B, H, n, d)) * scale)
    return K, V


# ---------------------------------------------------------------- sketch + norms

def test_hand_worked_example():
    """Alg. 1 (scoring and selection) on the exact-arithmetic example in tests/golden/hand_example.txt."""
    vals = {}
    with open(os.path.join(GOLDEN, "hand_example.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, *nums = line.split()
            vals[name] = np.array([float(x) for x in nums])
    K = bf16_bits([[[[1, 0], [0, 2], [1, 1], [3, -1]]]])
    V = bf16_bits([[[[2, 0], [1, 1], [0, 1], [1, 0]]]])
    G = np.array([[1, 1], [0, 2]], dtype=np.float32)
    sc, S, lK, lV = orc.score(K, V, G, return_factors=True)
    np.testing.assert_allclose(lK[0, 0], vals["lK"], rtol=0, atol=0)
    np.testing.assert_allclose(lV[0, 0], vals["lV"], rtol=0, atol=0)
    assert S[0, 0] == vals["sum"][0]
    np.testing.assert_allclose(sc[0, 0], vals["lKV"] / vals["sum"][0], rtol=1e-15)
    sck, Sk = orc.score(K, V, G, score_mode=1)
    scv, Sv = orc.score(K, V, G, score_mode=2)
    np.testing.assert_allclose(sck[0, 0], vals["lK"] / 38.0, rtol=1e-15)
    np.testing.assert_allclose(scv[0, 0], vals["lV"] / 24.0, rtol=1e-15)
    idx, cnt = orc.select_fixed(sc, budget=2, num_sink=1)
    assert idx[0, 0].tolist() == vals["select_s1_k2"].astype(int).tolist() and cnt[0, 0] == 2
    idx, cnt = orc.select_fixed(sc, budget=3, num_sink=1)
    assert idx[0, 0].tolist() == vals["select_s1_k3"].astype(int).tolist() and cnt[0, 0] == 3


def test_orthogonal_G_gives_exact_row_norms():
    """G orthogonal (r = d) => ||a G||^2 = ||a||^2 exactly (up to fp64 rounding)."""
    rng = np.random.default_rng(1)
    B, H, n, d = 2, 3, 17, 16
    K, V = rand_kv(rng, B, H, n, d)
    Q, _ = np.linalg.qr(rng.standard_normal((d, d)))
    # fp32 G: orthogonal to ~1e-7, so the identity holds to ~1e-6 relative
    for G in (np.eye(d, dtype=np.float32), Q.astype(np.float32)):
        _, _, lK, lV = orc.score(K, V, G, return_factors=True)
        nk = (synth.u16_to_f64(K) ** 2).sum(-1)
        nv = (synth.u16_to_f64(V) ** 2).sum(-1)
        np.testing.assert_allclose(lK, nk, rtol=2e-6)
        np.testing.assert_allclose(lV, nv, rtol=2e-6)


def test_selector_G_catches_transposed_or_misindexed_G():
    """G = [I_r; 0] picks the first r coordinates; one-hot G[t0][c0] = 2 gives 4 a[t0]^2.
    A transposed or mis-strided G changes both closed forms."""
    rng = np.random.default_rng(2)
    B, H, n, d, r = 1, 2, 9, 12, 5
    K, V = rand_kv(rng, B, H, n, d)
    Kd, Vd = synth.u16_to_f64(K), synth.u16_to_f64(V)
    G = np.zeros((d, r), dtype=np.float32)
    G[:r, :r] = np.eye(r)
    _, _, lK, lV = orc.score(K, V, G, return_factors=True)
    np.testing.assert_allclose(lK, (Kd[..., :r] ** 2).sum(-1), rtol=1e-14)
    np.testing.assert_allclose(lV, (Vd[..., :r] ** 2).sum(-1), rtol=1e-14)
    G = np.zeros((d, r), dtype=np.float32)
    G[7, 3] = 2.0
    _, _, lK, lV = orc.score(K, V, G, return_factors=True)
    np.testing.assert_allclose(lK, 4 * Kd[..., 7] ** 2, rtol=1e-14)
    np.testing.assert_allclose(lV, 4 * Vd[..., 7] ** 2, rtol=1e-14)


def test_per_head_G():
    """A [H, d, r] G applies head h's matrix to head h only."""
    rng = np.random.default_rng(3)
    B, H, n, d, r = 2, 3, 5, 8, 4
    K, V = rand_kv(rng, B, H, n, d)
    G = synth.make_G(d, r, seed=5, heads=H)
    sc, S = orc.score(K, V, G)
    for h in range(H):
        sh, Sh = orc.score(K[:, h:h + 1], V[:, h:h + 1], G[h])
        np.testing.assert_array_equal(sc[:, h], sh[:, 0])
        np.testing.assert_array_equal(S[:, h], Sh[:, 0])


def test_gaussian_sketch_moments():
    """G_ij ~ N(0,1/r) => l_j / ||a_j||^2 ~ chi2_r / r: mean 1, variance 2/r (Sec. 3.2)."""
    rng = np.random.default_rng(4)
    d, r, n, trials = 16, 8, 4, 2000
    K, V = rand_kv(rng, 1, 1, n, d)
    norms = (synth.u16_to_f64(K)[0, 0] ** 2).sum(-1)
    ratios = np.empty((trials, n))
    for t in range(trials):
        G = synth.make_G(d, r, seed=1000 + t)
        _, _, lK, _ = orc.score(K, V, G, return_factors=True)
        ratios[t] = lK[0, 0] / norms
    mean, var = ratios.mean(0), ratios.var(0)
    se_mean = np.sqrt(2.0 / r / trials)
    assert np.all(np.abs(mean - 1.0) < 4 * se_mean)
    # Var of the sample variance of chi2_r/r: (m4 - s^4)/T with m4 = 12(r+4)/r^3 + 4/r^2
    s2 = 2.0 / r
    m4 = 12.0 * (r + 4) / r ** 3 + s2 ** 2
    se_var = np.sqrt((m4 - s2 ** 2) / trials)
    assert np.all(np.abs(var - s2) < 4 * se_var)


def test_sketch_error_shrinks_like_inverse_sqrt_r():
    rng = np.random.default_rng(5)
    d, n = 32, 64
    K, V = rand_kv(rng, 1, 1, n, d)
    norms = (synth.u16_to_f64(K)[0, 0] ** 2).sum(-1)
    rs = [8, 32, 128, 512, 2048]
    errs = []
    for r in rs:
        e = []
        for seed in range(6):
            _, _, lK, _ = orc.score(K, V, synth.make_G(d, r, seed=seed), return_factors=True)
            e.append(np.sqrt(np.mean((lK[0, 0] / norms - 1.0) ** 2)))
        errs.append(np.mean(e))
    slope = np.polyfit(np.log(rs), np.log(errs), 1)[0]
    assert -0.62 < slope < -0.38, (slope, errs)
    np.testing.assert_allclose(errs, np.sqrt(2.0 / np.array(rs)), rtol=0.25)


def test_flat_spectrum_matches_svd_leverage():
    """On A = c U W^T (equal singular values) normalised sketch scores converge to the
    SVD row leverage ||U(j,:)||^2 / rank (Eq. row leverage score); sum of squared
    leverages equals rank(A)."""
    rng = np.random.default_rng(6)
    n, d, q = 48, 16, 16
    U, _ = np.linalg.qr(rng.standard_normal((n, q)))
    W, _ = np.linalg.qr(rng.standard_normal((d, q)))
    A = 3.0 * U @ W.T
    K = bf16_bits(A[None, None])
    Ad = synth.u16_to_f64(K)[0, 0]
    Us, sv, _ = np.linalg.svd(Ad, full_matrices=False)
    rank = int((sv > 1e-8 * sv[0]).sum())
    lev = (Us[:, :rank] ** 2).sum(-1)
    assert rank == q and abs(lev.sum() - rank) < 1e-9
    assert sv.max() / sv.min() < 1.02            # bf16 rounding keeps the spectrum ~flat
    errs = []
    for r in (16, 256, 4096):
        sc, _ = orc.score(K, K, synth.make_G(d, r, seed=r), score_mode=1)
        errs.append(np.abs(sc[0, 0] - lev / rank).max() / (lev / rank).max())
    assert errs[0] > errs[1] > errs[2] and errs[2] < 0.06, errs
    # exact limit: orthogonal G
    sc, _ = orc.score(K, K, np.eye(d, dtype=np.float32), score_mode=1)
    np.testing.assert_allclose(sc[0, 0], lev / rank, rtol=0.03)


def test_general_matrix_converges_to_row_norms_not_leverage():
    """Without whitening the sketch estimates squared row norms; on a matrix with a
    decaying spectrum these differ from SVD leverage (recorded, not a defect)."""
    rng = np.random.default_rng(7)
    n, d = 40, 8
    A = rng.standard_normal((n, d)) * np.array([8, 4, 2, 1, 1, 0.5, 0.25, 0.1])
    K = bf16_bits(A[None, None])
    Ad = synth.u16_to_f64(K)[0, 0]
    sc, _ = orc.score(K, K, synth.make_G(d, 8192, seed=0), score_mode=1)
    rown = (Ad ** 2).sum(-1)
    np.testing.assert_allclose(sc[0, 0], rown / rown.sum(), rtol=0.1)
    Us, _, _ = np.linalg.svd(Ad, full_matrices=False)
    lev = (Us ** 2).sum(-1) / d
    assert np.abs(sc[0, 0] - lev).max() > 0.2 * lev.max()


# ---------------------------------------------------------------- combine + normalise

def test_scores_sum_to_one_and_are_product_of_factors():
    rng = np.random.default_rng(8)
    B, H, n, d, r = 2, 4, 33, 16, 8
    K, V = rand_kv(rng, B, H, n, d)
    G = synth.make_G(d, r)
    sc, S, lK, lV = orc.score(K, V, G, return_factors=True)
    np.testing.assert_allclose(sc.sum(-1), 1.0, rtol=0, atol=1e-12)
    np.testing.assert_allclose(sc * S[..., None], lK * lV, rtol=1e-13)
    np.testing.assert_allclose(S, (lK * lV).sum(-1), rtol=1e-13)


def test_scale_invariance_and_permutation_equivariance():
    rng = np.random.default_rng(9)
    B, H, n, d, r = 1, 2, 21, 16, 8
    K, V = rand_kv(rng, B, H, n, d)
    G = synth.make_G(d, r)
    sc, S = orc.score(K, V, G)
    # powers of two scale bf16 values exactly
    K4 = bf16_bits(synth.u16_to_f64(K) * 4.0)
    Vh = bf16_bits(synth.u16_to_f64(V) * 0.5)
    sc2, S2 = orc.score(K4, Vh, G)
    np.testing.assert_allclose(sc2, sc, rtol=1e-13)
    np.testing.assert_allclose(S2, S * 16.0 * 0.25, rtol=1e-13)
    perm = rng.permutation(n)
    sc3, _ = orc.score(K[:, :, perm], V[:, :, perm], G)
    np.testing.assert_allclose(sc3, sc[:, :, perm], rtol=1e-12)
    i0, _ = orc.select_fixed(sc, budget=7)
    i3, _ = orc.select_fixed(sc3, budget=7)
    for h in range(H):
        assert sorted(perm[i3[0, h]].tolist()) == i0[0, h].tolist()


def test_ragged_lengths_ignore_padding_rows():
    rng = np.random.default_rng(10)
    B, H, n, d, r = 3, 2, 20, 8, 4
    K, V = rand_kv(rng, B, H, n, d)
    G = synth.make_G(d, r)
    lens = np.array([20, 7, 0], dtype=np.int32)
    sc, S = orc.score(K, V, G, seqlens=lens)
    for b in range(B):
        nb = lens[b]
        assert np.all(sc[b, :, nb:] == 0)
        if nb:
            ref, Sr = orc.score(K[b:b + 1, :, :nb], V[b:b + 1, :, :nb], G)
            np.testing.assert_array_equal(sc[b, :, :nb], ref[0])
        else:
            assert np.all(S[b] == 0)
    idx, cnt = orc.select_fixed(sc, budget=9, window=2, seqlens=lens)
    assert cnt[:, 0].tolist() == [9, 7, 0]
    assert idx[1, 0, :7].tolist() == list(range(7)) and np.all(idx[1, 0, 7:] == -1)
    assert np.all(idx[2] == -1)


def test_no_projection_ablation_is_plain_row_norms():
    rng = np.random.default_rng(11)
    K, V = rand_kv(rng, 1, 2, 10, 8)
    _, _, lK, lV = orc.score(K, V, synth.make_G(8, 4), use_projection=0, return_factors=True)
    np.testing.assert_allclose(lK, (synth.u16_to_f64(K) ** 2).sum(-1), rtol=1e-14)
    np.testing.assert_allclose(lV, (synth.u16_to_f64(V) ** 2).sum(-1), rtol=1e-14)


def test_planted_tokens_are_selected_cfg1_recipe():
    """Rows scaled x20 in K and V score ~1.6e5x typical, so every planted token outside
    the window is kept for any k >= 8 + window."""
    w = synth.shrink(synth.CONFIGS["cfg1"], n_max=256)
    K, V = synth.make_kv_element(w, 0)
    Ku, Vu = synth.to_u16(K)[None], synth.to_u16(V)[None]
    sc, _ = orc.score(Ku, Vu, synth.make_G(w.d, w.r))
    idx, cnt = orc.select_fixed(sc, budget=8 + 32, window=32)
    rown = (synth.u16_to_f64(Ku) ** 2).sum(-1)[0]
    for h in range(w.kv_heads):
        planted = np.argsort(rown[h])[-8:]
        assert rown[h][planted].min() > 100 * np.median(rown[h])
        assert set(planted.tolist()) <= set(idx[0, h].tolist())
        assert set(range(256 - 32, 256)) <= set(idx[0, h].tolist())


# ---------------------------------------------------------------- top-k

def brute_fixed(sc, k, s, w):
    n = len(sc)
    k_eff = min(k, n)
    forced = []
    for j in range(n - 1, max(n - w, 0) - 1, -1):
        if len(forced) < k_eff:
            forced.append(j)
    for j in range(min(s, n)):
        if j not in forced and len(forced) < k_eff:
            forced.append(j)
    cand = sorted((j for j in range(n) if j not in forced), key=lambda j: (-sc[j], j))
    return sorted(forced + cand[: k_eff - len(forced)])


@pytest.mark.parametrize("seed", range(6))
def test_select_fixed_matches_brute_force(seed):
    rng = np.random.default_rng(100 + seed)
    B, H, n = 2, 3, int(rng.integers(1, 40))
    sc = rng.random((B, H, n))
    if seed % 2:                                  # heavy ties
        sc = np.round(sc * 4) / 4
    k, s, w = int(rng.integers(0, n + 3)), int(rng.integers(0, 4)), int(rng.integers(0, 5))
    idx, cnt = orc.select_fixed(sc, budget=k, num_sink=s, window=w)
    for b in range(B):
        for h in range(H):
            want = brute_fixed(sc[b, h], k, s, w)
            c = cnt[b, h]
            assert c == len(want) == min(k, n)
            assert idx[b, h, :c].tolist() == want
            assert np.all(idx[b, h, c:] == -1)


def test_select_tie_rule_lower_index_wins():
    sc = np.array([[[0.1, 0.3, 0.3, 0.3, 0.0, 0.0]]])
    idx, _ = orc.select_fixed(sc, budget=2)
    assert idx[0, 0].tolist() == [1, 2]
    idx, _ = orc.select_fixed(sc, budget=5)
    assert idx[0, 0].tolist() == [0, 1, 2, 3, 4]
    idx, _ = orc.select_fixed(np.zeros((1, 1, 6)), budget=3, window=1)
    assert idx[0, 0].tolist() == [0, 1, 5]
    nan = np.array([[[np.nan, 0.5, np.nan, 0.25]]])
    idx, _ = orc.select_fixed(nan, budget=3)
    assert idx[0, 0].tolist() == [0, 1, 3]


def test_select_forced_set_and_budget_edges():
    rng = np.random.default_rng(12)
    sc = rng.random((1, 1, 30))
    idx, cnt = orc.select_fixed(sc, budget=10, num_sink=4, window=3)
    got = idx[0, 0].tolist()
    assert cnt[0, 0] == 10 and got == sorted(set(got))
    assert {0, 1, 2, 3, 27, 28, 29} <= set(got)
    # budget == |F|: nothing but forced tokens
    idx, _ = orc.select_fixed(sc, budget=7, num_sink=4, window=3)
    assert idx[0, 0].tolist() == [0, 1, 2, 3, 27, 28, 29]
    # budget < |F|: window first, then sinks
    idx, _ = orc.select_fixed(sc, budget=4, num_sink=4, window=3)
    assert idx[0, 0].tolist() == [0, 27, 28, 29]
    # budget >= n keeps everything
    idx, cnt = orc.select_fixed(sc, budget=64)
    assert cnt[0, 0] == 30 and idx[0, 0, :30].tolist() == list(range(30))
    # per-head budgets
    sc2 = rng.random((1, 3, 30))
    hb = np.array([[5, 0, 9]], dtype=np.int32)
    idx, cnt = orc.select_fixed(sc2, budget=9, head_budgets=hb)
    assert cnt[0].tolist() == [5, 0, 9]
    for h in range(3):
        assert idx[0, h, : hb[0, h]].tolist() == brute_fixed(sc2[0, h], hb[0, h], 0, 0)


# ---------------------------------------------------------------- AdaCurDKV

def brute_adaptive(sc, k, s, w, alpha):
    H, n = sc.shape
    k_eff = min(k, n)
    forced = brute_fixed(np.zeros(n), 0, 0, 0)
    forced = []
    for j in range(n - 1, max(n - w, 0) - 1, -1):
        if len(forced) < k_eff:
            forced.append(j)
    for j in range(min(s, n)):
        if j not in forced and len(forced) < k_eff:
            forced.append(j)
    p = min(max(int(np.floor(alpha * k)), len(forced)), k_eff)
    keep = [set(forced) for _ in range(H)]
    pool = []
    for h in range(H):
        cand = sorted((j for j in range(n) if j not in forced), key=lambda j: (-sc[h, j], j))
        keep[h] |= set(cand[: p - len(forced)])
        pool += [(-sc[h, j], h, j) for j in cand[p - len(forced):]]
    pool.sort()
    for _, h, j in pool[: H * (k_eff - p)]:
        keep[h].add(j)
    return [sorted(x) for x in keep]


@pytest.mark.parametrize("seed", range(6))
def test_select_adaptive_matches_brute_force(seed):
    rng = np.random.default_rng(200 + seed)
    B, H, n = 2, int(rng.integers(1, 5)), int(rng.integers(2, 40))
    sc = rng.random((B, H, n)) * rng.random((B, H, 1))      # heads with different mass
    if seed % 2:
        sc = np.round(sc * 8) / 8
    k, s, w = int(rng.integers(1, n + 2)), int(rng.integers(0, 3)), int(rng.integers(0, 4))
    alpha = float(rng.choice([0.0, 0.2, 0.5, 1.0]))
    idx, cnt, off = orc.select_adaptive(sc, budget=k, num_sink=s, window=w, alpha=alpha)
    assert off[0] == 0 and off[-1] == len(idx) == B * H * min(k, n)
    for b in range(B):
        want = brute_adaptive(sc[b], k, s, w, alpha)
        for h in range(H):
            o = off[b * H + h]
            assert cnt[b, h] == len(want[h]) == off[b * H + h + 1] - o
            assert idx[o:o + cnt[b, h]].tolist() == want[h]


def test_adaptive_invariants_and_special_cases():
    rng = np.random.default_rng(13)
    B, H, n, k, w = 2, 4, 64, 16, 3
    sc = rng.random((B, H, n)) * np.array([1.0, 0.1, 5.0, 0.01])[None, :, None]
    idx, cnt, off = orc.select_adaptive(sc, budget=k, window=w, alpha=0.2)
    assert np.all(cnt.sum(-1) == H * k)
    assert np.all(cnt >= max(int(np.floor(0.2 * k)), w))
    assert cnt[0, 2] > cnt[0, 0] > cnt[0, 1] >= cnt[0, 3]
    # alpha = 1 and H = 1 reduce to the fixed-budget selection
    fidx, fcnt = orc.select_fixed(sc, budget=k, window=w)
    idx1, cnt1, off1 = orc.select_adaptive(sc, budget=k, window=w, alpha=1.0)
    assert np.all(cnt1 == k) and idx1.tolist() == fidx.reshape(-1).tolist()
    one = sc[:, :1]
    fidx, _ = orc.select_fixed(one, budget=k, window=w)
    idx2, cnt2, _ = orc.select_adaptive(one, budget=k, window=w, alpha=0.2)
    assert idx2.tolist() == fidx.reshape(-1).tolist()
    # all the score mass in one head: it receives the whole pooled remainder
    sc3 = np.zeros((1, H, n))
    sc3[0, 1] = rng.random(n) + 1.0
    _, cnt3, _ = orc.select_adaptive(sc3, budget=k, window=w, alpha=0.25)
    p = max(int(np.floor(0.25 * k)), w)
    assert cnt3[0].tolist() == [p, p + H * (k - p), p, p]


# ---------------------------------------------------------------- gather, GQA, bytes

def test_compact_is_byte_exact_indexing():
    rng = np.random.default_rng(14)
    B, H, n, d = 2, 3, 25, 8
    K, V = rand_kv(rng, B, H, n, d)
    sc = rng.random((B, H, n))
    idx, cnt = orc.select_fixed(sc, budget=6, window=2)
    Ko, Vo = orc.compact(K, V, idx, cnt)
    for b in range(B):
        for h in range(H):
            np.testing.assert_array_equal(Ko[b, h], K[b, h, idx[b, h]])
            np.testing.assert_array_equal(Vo[b, h], V[b, h, idx[b, h]])
    pidx, pcnt, poff = orc.select_adaptive(sc, budget=6, window=2, alpha=0.2)
    Kp, Vp = orc.compact(K, V, pidx, pcnt, poff)
    for b in range(B):
        for h in range(H):
            o, c = poff[b * H + h], pcnt[b, h]
            np.testing.assert_array_equal(Kp[o:o + c], K[b, h, pidx[o:o + c]])
            np.testing.assert_array_equal(Vp[o:o + c], V[b, h, pidx[o:o + c]])


def test_gqa_group_map():
    assert [orc.kv_head_of_query(q, 32, 8) for q in (0, 3, 4, 31)] == [0, 0, 1, 7]
    assert [orc.kv_head_of_query(q, 8, 8) for q in range(8)] == list(range(8))


def test_cache_byte_accounting_matches_paper_128k_figure():
    """A 131072-token LLaMA-3.1-8B cache in bf16 is 16 GiB (the appendix's "approximately
    16 GB"); at 128,000 tokens the same formula gives 15.6 GiB (the main text's figure,
    Sec. 4.4)."""
    w = synth.CONFIGS["cfg4"]
    per_token = w.layers * w.batch * w.kv_heads * w.d * 2 * 2      # K and V, 2 bytes each
    assert per_token * w.n_max == 16 * 2 ** 30
    assert round(per_token * 128_000 / 2 ** 30, 1) == 15.6


# --------------------------------------------------------------------------- generation phase
def _history(B, H, N, d, seed, quantise=False):
    rng = np.random.default_rng(seed)
    K = rng.standard_normal((B, H, N, d)).astype(np.float32)
    V = rng.standard_normal((B, H, N, d)).astype(np.float32)
    if quantise:                       # few distinct rows -> many exactly equal scores
        K = np.round(K[:, :, :, :1] * 1.5) * np.ones((1, 1, 1, d), np.float32)
        V = np.ones_like(V)
    to_bits = lambda a: (a.view(np.uint32) >> 16).astype(np.uint16)     # truncation: still bf16 values
    return to_bits(np.ascontiguousarray(K)), to_bits(np.ascontiguousarray(V))


@pytest.mark.parametrize("quantise", [False, True])
@pytest.mark.parametrize("k,s,w", [(24, 4, 0), (24, 0, 8), (24, 2, 6), (10, 4, 6), (200, 4, 8)])
def test_generation_phase_equals_one_shot_selection(k, s, w, quantise):
    """Sec. 3.2 (method applies during generation): compressing incrementally, on any schedule,
    keeps exactly the tokens Alg. 1 keeps when applied once to the whole history."""
    from oracle import curdkv_decode_oracle as dec

    B, H, N, d, r = 2, 3, 150, 16, 8
    Ku, Vu = _history(B, H, N, d, seed=k + 7 * s + w, quantise=quantise)
    G = np.random.default_rng(1).standard_normal((d, r)).astype(np.float32) / np.sqrt(r)
    for schedule in ([40, 1, 1, 1, 30, 17, 60], [150], [1] * 150, [64, 64, 22]):
        cache = dec.CacheOracle(B, H, d)
        at = 0
        for step, t in enumerate(schedule):
            cache.append(Ku[:, :, at:at + t], Vu[:, :, at:at + t], G)
            at += t
            if step % 2 == 1 or at == N:            # compress now and then, and at the end
                cache.compress(k, s, w)
        assert at == N
        sc, _ = orc.score(Ku, Vu, G)
        idx, cnt = orc.select_fixed(sc, k, s, w)
        for b in range(B):
            for h in range(H):
                want = idx[b, h, : cnt[b, h]]
                np.testing.assert_array_equal(cache.pos[b][h], want)
                np.testing.assert_array_equal(cache.K[b][h], Ku[b, h, want])
                np.testing.assert_array_equal(cache.V[b][h], Vu[b, h, want])


def test_generation_phase_raw_scores_are_row_local():
    """A row's unnormalised score does not depend on which other rows are scored with it."""
    from oracle import curdkv_decode_oracle as dec

    Ku, Vu = _history(1, 2, 40, 16, seed=3)
    G = np.random.default_rng(2).standard_normal((16, 8)).astype(np.float32)
    full = dec.raw_scores(Ku, Vu, G)
    part = dec.raw_scores(Ku[:, :, 10:25], Vu[:, :, 10:25], G)
    np.testing.assert_array_equal(full[:, :, 10:25], part)
    sc, S = orc.score(Ku, Vu, G)
    np.testing.assert_allclose(full / S[..., None], sc, rtol=1e-14)


# --------------------------------------------------------------------------- whitened sketch
def test_whitened_scores_are_exact_leverage_for_identity_G():
    """Eq. (row leverage score): with G = I and no ridge, ||a_j L^-T||^2 = ||U(j,:)||^2 (numpy SVD),
    the scores sum to rank(A) = d, and they ignore any invertible mixing of the columns."""
    from oracle import curdkv_whiten_oracle as wh

    rng = np.random.default_rng(0)
    n, d = 300, 24
    A = rng.standard_normal((n, d)) * np.exp(rng.standard_normal((1, d)) * 2.0)   # badly scaled columns
    lev = wh.whitened_row_scores(A, np.eye(d), 0.0)
    U = np.linalg.svd(A, full_matrices=False)[0]
    np.testing.assert_allclose(lev, np.sum(U * U, axis=1), rtol=1e-9)
    np.testing.assert_allclose(lev.sum(), d, rtol=1e-10)
    T = rng.standard_normal((d, d)) + 3 * np.eye(d)
    np.testing.assert_allclose(wh.whitened_row_scores(A @ T, np.eye(d), 0.0), lev, rtol=1e-7)
    # the plain sketch of Alg. 1 is NOT invariant to such mixing: it follows the row norms
    plain = np.sum(A * A, axis=1)
    assert np.corrcoef(plain / plain.sum(), lev / lev.sum())[0, 1] < 0.9


def test_whitened_sketch_is_unbiased_and_converges():
    """Gaussian G ~ N(0, 1/r): E ||a_j W||^2 = leverage; the error shrinks like r^-1/2."""
    from oracle import curdkv_whiten_oracle as wh

    rng = np.random.default_rng(1)
    n, d = 200, 16
    A = rng.standard_normal((n, d)) @ np.diag(np.linspace(1, 30, d))
    exact = wh.whitened_row_scores(A, np.eye(d), 0.0)
    r = 8
    draws = np.stack([wh.whitened_row_scores(A, rng.standard_normal((d, r)) / np.sqrt(r), 0.0)
                      for _ in range(1500)])
    sigma = exact * np.sqrt(2.0 / r) / np.sqrt(draws.shape[0])       # chi-square: var = 2 l^2 / r
    assert np.all(np.abs(draws.mean(0) - exact) < 4.5 * sigma)
    errs = []
    for r in (8, 128, 2048):
        G = rng.standard_normal((d, r)) / np.sqrt(r)
        errs.append(np.median(np.abs(wh.whitened_row_scores(A, G, 0.0) - exact) / exact))
    assert errs[0] > 2.5 * errs[1] > 6 * errs[2]


def test_whitened_ridge_matches_direct_inverse_and_short_sequences():
    from oracle import curdkv_whiten_oracle as wh

    rng = np.random.default_rng(2)
    n, d = 40, 16
    A = rng.standard_normal((n, d))
    ridge = 1e-2
    lam = ridge * np.trace(A.T @ A) / d
    want = np.einsum("ij,jk,ik->i", A, np.linalg.inv(A.T @ A + lam * np.eye(d)), A)
    np.testing.assert_allclose(wh.whitened_row_scores(A, np.eye(d), ridge), want, rtol=1e-10)
    assert np.all(want < wh.whitened_row_scores(A, np.eye(d), 0.0))
    # fewer rows than columns: the Gram matrix is singular, the ridge keeps the factorisation defined
    short = wh.whitened_row_scores(A[:5], np.eye(d), ridge)
    assert np.all(np.isfinite(short)) and np.all(short > 0) and np.all(short < 1)


def test_whitened_pipeline_normalises_and_respects_lengths():
    from oracle import curdkv_whiten_oracle as wh

    rng = np.random.default_rng(3)
    B, H, n, d, r = 2, 2, 64, 16, 8
    to_bits = lambda a: (np.ascontiguousarray(a, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16)
    K, V = to_bits(rng.standard_normal((B, H, n, d))), to_bits(rng.standard_normal((B, H, n, d)))
    G = (rng.standard_normal((d, r)) / np.sqrt(r)).astype(np.float32)
    lens = np.array([64, 37], np.int32)
    sc, S, lK, lV = wh.score_whitened(K, V, G, 1e-4, seqlens=lens)
    np.testing.assert_allclose(sc.sum(-1), 1.0, rtol=1e-12)
    assert np.all(sc[1, :, 37:] == 0)
    np.testing.assert_allclose(sc * S[..., None], lK * lV, rtol=1e-12)
    sc2, _, _, _ = wh.score_whitened(K[1:, :, :37], V[1:, :, :37], G, 1e-4)
    np.testing.assert_allclose(sc2[0], sc[1, :, :37], rtol=1e-12)


# --------------------------------------------------------------------------- eviction loss
def test_attention_oracle_closed_forms():
    from oracle import curdkv_eviction_oracle as ev

    rng = np.random.default_rng(0)
    m, n, d = 7, 50, 16
    Q, K, V = rng.standard_normal((m, d)), rng.standard_normal((n, d)), rng.standard_normal((n, d))
    # all keys equal -> uniform weights -> every output row is the mean value row
    O = ev.attention_out(Q, np.tile(K[:1], (n, 1)), V)
    np.testing.assert_allclose(O, np.tile(V.mean(0), (m, 1)), rtol=1e-12)
    # softmax rows sum to one: constant values come back unchanged
    np.testing.assert_allclose(ev.attention_out(Q, K, np.ones((n, d))), 1.0, rtol=1e-12)
    # one key aligned with a query and scaled up takes all the weight of that query
    K2 = K.copy()
    K2[13] = 40.0 * Q[3] / np.linalg.norm(Q[3])
    np.testing.assert_allclose(ev.attention_out(Q, K2, V)[3], V[13], atol=1e-9)
    # shifting every key by one vector shifts each row's logits by a constant: no change
    np.testing.assert_allclose(ev.attention_out(Q, K + rng.standard_normal((1, d)), V),
                               ev.attention_out(Q, K, V), rtol=1e-9)
    # explicit two-key case
    q, k0, k1 = np.array([[1.0, 0.0]]), np.array([2.0, 0.0]), np.array([0.0, 5.0])
    w0 = np.exp(2.0) / (np.exp(2.0) + 1.0)
    got = ev.attention_out(q, np.stack([k0, k1]), np.array([[1.0, 0.0], [0.0, 1.0]]))
    np.testing.assert_allclose(got, [[w0, 1 - w0]], rtol=1e-13)
    # scale multiplies the logits
    np.testing.assert_allclose(ev.attention_out(Q, K, V, scale=0.25), ev.attention_out(0.25 * Q, K, V),
                               rtol=1e-12)


def test_eviction_loss_properties_and_lemma1():
    """Lemma 1: ||softmax(QK^T)V - softmax(QK'^T)V'||_F <= sqrt(n)||V - V'||_F + 2 sqrt(n)||V'||_F with
    zeroed rows; keeping everything loses nothing; zeroed rows are keys with logit 0 and value 0."""
    from oracle import curdkv_eviction_oracle as ev

    rng = np.random.default_rng(1)
    n, d = 60, 16
    Q, K, V = rng.standard_normal((n, d)), rng.standard_normal((n, d)), rng.standard_normal((n, d))
    assert ev.eviction_loss(Q, K, V, np.arange(n))[0] < 1e-12
    assert ev.eviction_loss(Q, K, V, np.arange(n), zeroed=True)[0] < 1e-12
    for k in (1, 5, 30, 59):
        kept = np.sort(rng.choice(n, size=k, replace=False))
        loss0, ref = ev.eviction_loss(Q, K, V, kept, zeroed=True)
        assert loss0 <= ev.lemma1_bound(V, kept)
        # the zeroed form is attention over the full-size K', V'
        Kp, Vp = np.zeros_like(K), np.zeros_like(V)
        Kp[kept], Vp[kept] = K[kept], V[kept]
        direct = np.linalg.norm(ev.attention_out(Q, K, V) - ev.attention_out(Q, Kp, Vp))
        np.testing.assert_allclose(loss0, direct, rtol=1e-10)
        np.testing.assert_allclose(ref, np.linalg.norm(ev.attention_out(Q, K, V)), rtol=1e-13)
    # evicting rows whose value is zero and whose key repels every query costs (almost) nothing
    K3, V3 = K.copy(), V.copy()
    K3[40:] = -50.0 * np.sign(Q.sum(0, keepdims=True))
    Qpos = np.abs(Q) * np.sign(Q.sum(0, keepdims=True))
    V3[40:] = 0.0
    assert ev.eviction_loss(Qpos, K3, V3, np.arange(40))[0] < 1e-9


def test_lemma1_bound_hand_worked_values():
    """The bound of Lemma 1, sqrt(n)||V - V'||_F + 2 sqrt(n)||V'||_F, on value matrices whose norms
    are whole numbers (tests/golden/lemma1_example.txt): catches a dropped factor 2, a dropped term,
    n in place of sqrt(n), and V' built from the evicted instead of the kept rows."""
    from oracle import curdkv_eviction_oracle as ev

    rows = np.array([[3.0, 0.0], [0.0, 4.0], [12.0, 0.0]])
    cases = 0
    for line in open(os.path.join(GOLDEN, "lemma1_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        n, kept, bound = line.split()
        n = int(n)
        kept = [] if kept == "-" else [int(t) for t in kept.split(",")]
        V = np.zeros((n, 2))
        V[:3] = rows
        assert ev.lemma1_bound(V, kept) == pytest.approx(float(bound), rel=1e-15, abs=0)
        cases += 1
    assert cases == 7


def test_generation_phase_ragged_appends_equal_dense_appends():
    """CacheOracle.append with t_new: blocks in which sequence b brings only t_new[b] real rows (the
    rest of the block is padding) must leave exactly the state that appending the real rows alone
    leaves -- positions count real rows only, padding rows never enter -- and the final kept set
    must be that of one application of Alg. 1 to each sequence's real history."""
    from oracle import curdkv_decode_oracle as dec

    rng = np.random.default_rng(5)
    B, H, d, r, t = 3, 2, 16, 8, 12
    G = (rng.standard_normal((d, r)) / np.sqrt(r)).astype(np.float32)
    k, s, w = 14, 2, 3
    t_news = [np.array(v) for v in ([12, 5, 0], [0, 12, 7], [3, 1, 12], [12, 12, 12], [1, 0, 2], [9, 4, 0])]
    ragged = dec.CacheOracle(B, H, d)
    dense = [dec.CacheOracle(1, H, d) for _ in range(B)]
    hist_K = [[] for _ in range(B)]
    hist_V = [[] for _ in range(B)]
    for step, tn in enumerate(t_news):
        Kb, Vb = rand_kv(rng, B, H, t, d)
        ragged.append(Kb, Vb, G, tn)
        for b in range(B):
            tb = int(tn[b])
            hist_K[b].append(Kb[b:b + 1, :, :tb])
            hist_V[b].append(Vb[b:b + 1, :, :tb])
            if tb:                                        # the same real rows, as a full block
                dense[b].append(Kb[b:b + 1, :, :tb], Vb[b:b + 1, :, :tb], G)
        if step in (2, 4):
            ragged.compress(k, s, w)
            for b in range(B):
                dense[b].compress(k, s, w)
    ragged.compress(k, s, w)
    totals = np.sum(t_news, axis=0)
    np.testing.assert_array_equal(ragged.total, totals)
    for b in range(B):
        dense[b].compress(k, s, w)
        assert dense[b].total[0] == totals[b]
        Kh, Vh = np.concatenate(hist_K[b], axis=2), np.concatenate(hist_V[b], axis=2)
        sc, _ = orc.score(Kh, Vh, G)
        idx, cnt = orc.select_fixed(sc, k, s, w)
        for h in range(H):
            np.testing.assert_array_equal(ragged.pos[b][h], dense[b].pos[0][h])
            np.testing.assert_array_equal(ragged.raw[b][h], dense[b].raw[0][h])
            np.testing.assert_array_equal(ragged.K[b][h], dense[b].K[0][h])
            np.testing.assert_array_equal(ragged.V[b][h], dense[b].V[0][h])
            one_shot = idx[0, h, : cnt[0, h]]
            np.testing.assert_array_equal(ragged.pos[b][h], one_shot)
            np.testing.assert_array_equal(ragged.K[b][h], Kh[0, h][one_shot])
