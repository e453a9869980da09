"""Comparison rules between the CUDA path and the fp64 oracle.

Scores: |gpu - oracle| <= 1e-3 * oracle + 1e-6 * max_j oracle_j  (fp32 accumulation).
Indices: exact wherever the oracle's score gap at the cut exceeds 1e-4 relative:
with T = oracle score of the weakest selected candidate, every candidate above
T(1+1e-4) must be selected and none below T(1-1e-4); the set has exactly the
oracle's size, is sorted, distinct, in range and contains the forced tokens.
"""
import numpy as np

SCORE_RTOL = 1e-3
SCORE_ATOL_FRAC = 1e-6
TIE_BAND = 1e-4


def assert_scores_close(gpu, ref, what=""):
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert gpu.shape == ref.shape, (gpu.shape, ref.shape)
    assert np.all(np.isfinite(gpu)), f"{what}: non-finite GPU scores"
    tol = SCORE_RTOL * np.abs(ref) + SCORE_ATOL_FRAC * np.abs(ref).max(axis=-1, keepdims=True)
    err = np.abs(gpu - ref)
    bad = err > tol
    if bad.any():
        i = np.unravel_index(np.argmax(err - tol), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} scores outside tolerance; worst at {i}: "
                             f"gpu={gpu[i]:.9g} ref={ref[i]:.9g}")
    with np.errstate(divide="ignore", invalid="ignore"):
        rel = np.where(ref > 0, err / ref, 0.0)
    return float(rel.max())


def forced_tokens(n, k_eff, s, w):
    forced = []
    for j in range(n - 1, max(n - w, 0) - 1, -1):
        if len(forced) < k_eff:
            forced.append(j)
    for j in range(min(s, n)):
        if j not in forced and len(forced) < k_eff:
            forced.append(j)
    return set(forced)


def assert_selection_within_band(gpu_idx, ref_idx, ref_scores, n, forced, what=""):
    """One head.  gpu_idx / ref_idx: 1-D arrays of the kept token indices (no -1 tail)."""
    g = np.asarray(gpu_idx, dtype=np.int64)
    r = np.asarray(ref_idx, dtype=np.int64)
    assert len(g) == len(r), f"{what}: kept {len(g)} rows, oracle kept {len(r)}"
    if len(g) == 0:
        return 0
    assert g.min() >= 0 and g.max() < n, f"{what}: index out of range"
    assert np.all(np.diff(g) > 0), f"{what}: indices not strictly ascending"
    gs, rs = set(g.tolist()), set(r.tolist())
    assert forced <= gs, f"{what}: forced tokens missing"
    if gs == rs:
        return 0
    sel_cand = [j for j in r.tolist() if j not in forced]
    T = min(ref_scores[j] for j in sel_cand) if sel_cand else 0.0
    for j in gs - rs:       # GPU kept, oracle dropped: must lie inside the band
        assert ref_scores[j] >= T * (1 - TIE_BAND), f"{what}: token {j} kept but scores below the cut"
    for j in rs - gs:       # oracle kept, GPU dropped
        assert ref_scores[j] <= T * (1 + TIE_BAND), f"{what}: token {j} dropped but scores above the cut"
    return len(gs ^ rs)


def assert_adaptive_within_band(gpu_idx, gpu_off, ref_idx, ref_off, ref_scores, b, H, n, s, w, what=""):
    """AdaCurDKV, the heads of one (layer, sequence) b.  gpu_idx / ref_idx are the packed index
    arrays with their offsets; ref_scores [H, n] the oracle's scores of this b.  Every head keeps
    sorted, distinct, in-range indices containing its forced tokens, the layer total equals the
    oracle's, and a token on which the two disagree scores within the tie band of one of the two
    cuts that can decide it: its own head's weakest kept candidate (the safeguard cut, or the
    layer-wide cut where that lies lower) or the weakest kept candidate of the whole layer."""
    ref_scores = np.asarray(ref_scores)
    cuts, sets = [], []
    for h in range(H):
        g = np.asarray(gpu_idx[gpu_off[b * H + h]: gpu_off[b * H + h + 1]], dtype=np.int64)
        r = np.asarray(ref_idx[ref_off[b * H + h]: ref_off[b * H + h + 1]], dtype=np.int64)
        if len(g):
            assert g.min() >= 0 and g.max() < n, f"{what} h={h}: index out of range"
            assert np.all(np.diff(g) > 0), f"{what} h={h}: indices not strictly ascending"
        forced = forced_tokens(n, min(len(r), len(g)), s, w)
        assert forced <= set(g.tolist()), f"{what} h={h}: forced tokens missing"
        cand = [j for j in r.tolist() if j not in forced]
        cuts.append(min(ref_scores[h][j] for j in cand) if cand else np.inf)
        sets.append((set(g.tolist()), set(r.tolist())))
    assert sum(len(g) for g, _ in sets) == sum(len(r) for _, r in sets), f"{what}: layer totals differ"
    lo_cut = min(cuts)
    diffs = 0
    for h, (g, r) in enumerate(sets):
        for j in g ^ r:
            rel = min(abs(ref_scores[h][j] / c - 1.0) for c in (lo_cut, cuts[h]) if np.isfinite(c) and c > 0)
            assert rel < TIE_BAND, f"{what} h={h}: token {j} differs {rel:.3g} away from a cut"
            diffs += 1
    return diffs
