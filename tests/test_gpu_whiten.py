"""Whitened sketch (approximate leverage scores, Eq. row-leverage) on the GPU against the fp64
oracle.  Needs a B200."""
import numpy as np
import pytest
import torch

from oracle import curdkv_oracle as orc
from oracle import curdkv_whiten_oracle as wh
from paper_2509_15038_b200 import binding as cur
from paper_2509_15038_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu
DEV = "cuda"
# fp32 Gram accumulation over n rows feeds a Cholesky whose error grows with the conditioning of
# A^T A + lambda I; for the synthetic caches (condition number ~1e2-1e4) the scores stay within
# 2e-3 of the fp64 oracle
WHITEN_RTOL = 2e-3


def _score(K, V, G, ridge, seqlens=None):
    sl = None if seqlens is None else torch.as_tensor(seqlens, dtype=torch.int32, device=DEV)
    Gd = torch.as_tensor(G, dtype=torch.float32, device=DEV).contiguous()
    desc = cur.make_desc(K, V, G.shape[-1], seqlens=sl, whiten=1, ridge=ridge)
    ws = cur.alloc_workspace(desc)
    scores, sums = cur.curdkv_score(K, V, Gd, desc, ws)
    flags = cur.curdkv_device_status(ws)
    return desc, ws, scores, sums, flags


def _check(K, V, G, ridge, seqlens=None, what=""):
    desc, ws, scores, sums, flags = _score(K, V, G, ridge, seqlens)
    assert flags == 0, f"{what}: device flags {flags:#x}"
    rs, rS, _, _ = wh.score_whitened(synth.to_u16(K), synth.to_u16(V), G, ridge, seqlens=seqlens)
    got = scores.cpu().numpy().astype(np.float64)
    tol = WHITEN_RTOL * rs + 1e-6 * rs.max(-1, keepdims=True)
    err = np.abs(got - rs)
    assert np.all(np.isfinite(got))
    assert np.all(err <= tol), f"{what}: worst rel err {np.max(err / np.maximum(rs, 1e-300)):.3e}"
    np.testing.assert_allclose(sums.cpu().numpy(), rS, rtol=WHITEN_RTOL)
    np.testing.assert_allclose(got.sum(-1)[rS > 0], 1.0, rtol=1e-4)
    return desc, ws, scores, rs


@pytest.mark.parametrize("r", [32, 64, 20])
def test_whitened_scores_match_oracle(r):
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=2, n_max=1536, kv_heads=3, q_heads=3)
    K, V, _ = synth.make_kv(w, DEV)
    _check(K, V, synth.make_G(w.d, r, seed=r), 1e-4, what=f"r={r}")


def test_whitened_long_rows_and_selection():
    """Several segments per head, rows far beyond one tile; selection on the whitened scores."""
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=1, n_max=8192, kv_heads=2, q_heads=2)
    K, V, _ = synth.make_kv(w, DEV)
    G = synth.make_G(w.d, 32, seed=0)
    desc, ws, scores, rs = _check(K, V, G, 1e-4, what="long")
    idx, cnt, _ = cur.curdkv_select(scores, desc, 900, num_sink=4, window=64, workspace=ws)
    eidx, ecnt = orc.select_fixed(scores.cpu().numpy().astype(np.float64), 900, num_sink=4, window=64)
    np.testing.assert_array_equal(idx.cpu().numpy(), eidx)
    # whitening removes the pull of the outlier channels: the kept set differs from plain Alg. 1
    d0 = cur.make_desc(K, V, 32)
    s0, _ = cur.curdkv_score(K, V, torch.as_tensor(G, device=DEV), d0, cur.alloc_workspace(d0))
    i0, _, _ = cur.curdkv_select(s0, d0, 900, num_sink=4, window=64)
    assert (i0 != idx).any()


def test_whitened_full_length_rows_r64():
    """Rows as long as the benchmark's (32768 tokens: many tiles per segment), 64 sketch columns."""
    w = synth.shrink(synth.CONFIGS["cfg3"], layers=1, batch=1, kv_heads=2, q_heads=2)
    K, V, _ = synth.make_kv(w, DEV)
    _check(K, V, synth.make_G(w.d, 64, seed=2), 1e-4, what="n=32768 r=64")


def test_whitened_ragged_and_odd_lengths():
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=1, batch=5, n_max=1000, kv_heads=2, q_heads=2)
    K, V, _ = synth.make_kv(w, DEV)
    G = synth.make_G(w.d, 32, seed=1)
    lens = np.array([1000, 777, 130, 0, 50], dtype=np.int32)      # 50 < d: only the ridge keeps M definite
    _check(K, V, G, 1e-3, seqlens=lens, what="ragged")


def test_whitened_identity_G_gives_svd_leverage():
    """G = first 64 coordinates: l^K_j = ||a_j L^-T[:, :64]||^2; with V = K the product is its square.
    Checked against numpy's SVD on the same bits (r = d is beyond the kernel's 64 columns, so the
    comparison uses the oracle's W restricted to 64 columns and the SVD identity for its full sum)."""
    n, d = 640, 128
    g = torch.Generator(device=DEV).manual_seed(3)
    K = (torch.randn((1, 1, n, d), generator=g, device=DEV) *
         torch.exp(torch.randn((1, 1, 1, d), generator=g, device=DEV))).to(torch.bfloat16)
    G = np.zeros((d, 64), dtype=np.float32)
    G[:64, :64] = np.eye(64)
    desc, ws, scores, sums, flags = _score(K, K, G, 0.0)
    assert flags == 0
    A = synth.u16_to_f64(synth.to_u16(K))[0, 0]
    L = np.linalg.cholesky(A.T @ A)
    Y = A @ np.linalg.inv(L).T[:, :64]
    lk = np.sum(Y * Y, axis=1)
    want = lk * lk / np.sum(lk * lk)
    pu.assert_scores_close(scores.cpu().numpy()[0, 0], want, "identity G")
    U = np.linalg.svd(A, full_matrices=False)[0]
    full = np.sum((A @ np.linalg.inv(L).T) ** 2, axis=1)
    np.testing.assert_allclose(full, np.sum(U * U, axis=1), rtol=1e-8)


def test_whitened_and_attention_on_token_major_views():
    """K, V stored [B, n, H, d] and viewed as [B, H, n, d]: strides reach the Gram, the per-item
    sketch and the attention kernels through their tensor maps."""
    from oracle import curdkv_eviction_oracle as ev

    B, H, n, d = 2, 3, 700, 128
    g = torch.Generator(device=DEV).manual_seed(17)
    Kb = torch.randn((B, n, H, d), generator=g, device=DEV).to(torch.bfloat16)
    Vb = torch.randn((B, n, H, d), generator=g, device=DEV).to(torch.bfloat16)
    K, V = Kb.permute(0, 2, 1, 3), Vb.permute(0, 2, 1, 3)
    _check(K, V, synth.make_G(d, 32, seed=4), 1e-4, what="token-major whitened")
    Q = torch.randn((B, H, 96, d), generator=g, device=DEV).to(torch.bfloat16)
    desc = cur.make_desc(K, V, 32)
    O, ws = cur.curdkv_attention_out(Q, K, V, desc, scale=0.1)
    assert cur.curdkv_device_status(ws) == 0
    got = O.cpu().numpy().astype(np.float64)
    f = lambda t: synth.u16_to_f64(synth.to_u16(t))
    Qf, Kf, Vf = f(Q), f(K), f(V)
    for b in range(B):
        for h in range(H):
            want = ev.attention_out(Qf[b, h], Kf[b, h], Vf[b, h], 0.1)
            assert np.abs(got[b, h] - want).max() <= 2e-4 * np.abs(want).max()


def test_whitened_rejects_unsupported_shapes():
    K = torch.zeros((1, 1, 64, 128), dtype=torch.bfloat16, device=DEV)
    G = torch.zeros((128, 32), dtype=torch.float32, device=DEV)
    desc = cur.make_desc(K, K, 32, whiten=1, ridge=1e-4)
    with pytest.raises(cur.CurdkvError):
        cur.curdkv_score(K, K, G, desc, cur.alloc_workspace(desc))
    desc = cur.make_desc(K, K, 32, whiten=1, ridge=-1.0)
    with pytest.raises((cur.CurdkvError, ValueError)):
        cur.curdkv_score(K, K, G, desc, torch.zeros(1 << 20, dtype=torch.uint8, device=DEV))


def test_singular_gram_matrix_is_flagged_not_faulted():
    """Channels that are zero in every row make the Gram matrix singular: without a ridge the
    factorisation meets a zero pivot and raises the NOT_SPD bit of the status word (the results of
    that call are void); with the ridge the same input is scored normally."""
    g = torch.Generator(device=DEV).manual_seed(9)
    K = torch.randn((1, 2, 1024, 128), generator=g, device=DEV)
    K[..., 5] = 0.0
    K[..., 77] = 0.0
    K = K.to(torch.bfloat16)
    V = torch.randn((1, 2, 1024, 128), generator=g, device=DEV).to(torch.bfloat16)
    G = torch.as_tensor(synth.make_G(128, 32, seed=1), device=DEV)
    desc = cur.make_desc(K, V, 32, whiten=1, ridge=0.0)
    ws = cur.alloc_workspace(desc)
    cur.curdkv_score(K, V, G, desc, ws)
    torch.cuda.synchronize()
    assert cur.curdkv_device_status(ws) & cur.DEV_NOT_SPD
    desc = cur.make_desc(K, V, 32, whiten=1, ridge=1e-4)
    ws = cur.alloc_workspace(desc)
    scores, sums = cur.curdkv_score(K, V, G, desc, ws)
    assert cur.curdkv_device_status(ws) == 0
    assert bool(torch.isfinite(scores).all())
    assert torch.allclose(scores.sum(-1), torch.ones_like(scores.sum(-1)), atol=1e-4)
