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
