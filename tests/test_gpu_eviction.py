"""Eviction-loss evaluator on the GPU (attention output of the full and the compressed cache,
through the C ABI) against the fp64 oracle.  Needs a B200."""
import numpy as np
import pytest
import torch

from oracle import curdkv_eviction_oracle as ev
from paper_2509_15038_b200 import binding as cur
from paper_2509_15038_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"
# exp2 of fp32 logits and bf16 (hi + lo) weights: outputs agree with fp64 to ~1e-5 of the largest
# entry; 2e-4 leaves room for logits of a few hundred
OUT_TOL = 2e-4


def _f64(t):
    return synth.u16_to_f64(synth.to_u16(t))


def _queries(B, H, m, d, seed, gain=1.0):
    g = torch.Generator(device=DEV).manual_seed(seed)
    return (gain * torch.randn((B, H, m, d), generator=g, device=DEV)).to(torch.bfloat16)


def _check_out(O, Q, K, V, lens, scale, extra=None, what="", tol=OUT_TOL):
    got = O.cpu().numpy().astype(np.float64)
    Qf, Kf, Vf = _f64(Q), _f64(K), _f64(V)
    B, H = Q.shape[:2]
    for b in range(B):
        for h in range(H):
            n = int(lens[b, h])
            if n == 0:
                assert np.all(got[b, h] == 0)
                continue
            want = ev.attention_out(Qf[b, h], Kf[b, h, :n], Vf[b, h, :n], scale,
                                    0 if extra is None else int(extra[b, h]))
            err = np.abs(got[b, h] - want).max()
            assert err <= tol * np.abs(want).max(), f"{what} b={b} h={h}: err {err:.3e}"


@pytest.mark.parametrize("scale", [1.0 / np.sqrt(128.0), 1.0])
def test_attention_out_matches_oracle(scale):
    """Ragged key counts incl. 0, 1 and non-multiples of the tile; query rows not a multiple of 128."""
    B, H, n, d, m = 3, 2, 1000, 128, 200
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=1, batch=B, n_max=n, kv_heads=H, q_heads=H)
    K, V, _ = synth.make_kv(w, DEV)
    Q = _queries(B, H, m, d, seed=5, gain=0.5 if scale == 1.0 else 1.0)
    lens = np.array([1000, 333, 0], dtype=np.int32)
    desc = cur.make_desc(K, V, 32, seqlens=torch.as_tensor(lens, device=DEV))
    O, ws = cur.curdkv_attention_out(Q, K, V, desc, scale=scale)
    assert cur.curdkv_device_status(ws) == 0
    _check_out(O, Q, K, V, np.repeat(lens[:, None], H, 1), scale, what=f"scale={scale:.3f}")
    # explicit per-head row counts override the sequence lengths
    rows = np.array([[1, 129], [128, 999], [7, 0]], dtype=np.int32)
    O, ws = cur.curdkv_attention_out(Q, K, V, desc, scale=scale,
                                     head_rows=torch.as_tensor(rows.reshape(-1), device=DEV))
    assert cur.curdkv_device_status(ws) == 0
    _check_out(O, Q, K, V, rows, scale, what="head_rows")
    # single bf16 weights (one product per tile instead of two): bf16 rounding of the weights, 2^-9
    # relative each, averages out over the keys; 4e-3 of the largest entry is the documented bound
    O1, ws = cur.curdkv_attention_out(Q, K, V, desc, scale=scale, weight_split=False,
                                      head_rows=torch.as_tensor(rows.reshape(-1), device=DEV))
    assert cur.curdkv_device_status(ws) == 0
    _check_out(O1, Q, K, V, rows, scale, what="single bf16 weights", tol=4e-3)
    assert not torch.equal(O1, O)


def test_constant_values_and_nan_padding():
    """Softmax rows sum to one (V = 1 comes back as 1), and NaNs in the padding rows never leak."""
    B, H, n, d, m = 1, 2, 300, 128, 64
    g = torch.Generator(device=DEV).manual_seed(1)
    K = torch.randn((B, H, n, d), generator=g, device=DEV).to(torch.bfloat16)
    V = torch.ones((B, H, n, d), device=DEV).to(torch.bfloat16)
    K[:, :, 200:] = float("nan")
    V[:, :, 200:] = float("nan")
    Q = _queries(B, H, m, d, seed=2)
    desc = cur.make_desc(K, V, 32, seqlens=torch.tensor([200], dtype=torch.int32, device=DEV))
    O, ws = cur.curdkv_attention_out(Q, K, V, desc, scale=0.1)
    assert cur.curdkv_device_status(ws) == 0
    np.testing.assert_allclose(O.cpu().numpy(), 1.0, rtol=1e-5)


@pytest.mark.parametrize("adaptive", [False, True])
def test_eviction_loss_of_a_curdkv_selection(adaptive):
    """score -> select -> compact -> attention on both caches -> loss, against the oracle's loss for
    the rows the GPU kept; also Lemma 1's zeroed form and its bound."""
    B, H, n, d, m, k = 2, 4, 2048, 128, 256, 300
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=1, batch=B, n_max=n, kv_heads=H, q_heads=H, data_seed=9)
    K, V, _ = synth.make_kv(w, DEV)
    Q = _queries(B, H, m, d, seed=3)
    scale = 1.0 / np.sqrt(d)
    G = torch.as_tensor(synth.make_G(d, 32, seed=0), device=DEV)
    desc = cur.make_desc(K, V, 32)
    ws = cur.alloc_workspace(desc, k, adaptive)
    scores, _ = cur.curdkv_score(K, V, G, desc, ws)
    idx, cnt, off = cur.curdkv_select(scores, desc, k, num_sink=4, window=32, adaptive=adaptive, workspace=ws)
    Kc, Vc = cur.curdkv_compact(K, V, desc, idx, cnt, off, packed=adaptive, workspace=ws)
    O, _ = cur.curdkv_attention_out(Q, K, V, desc, scale=scale)
    rows = cnt.reshape(-1).contiguous()
    if adaptive:
        Oc, aws = cur.curdkv_attention_out(Q, Kc, Vc, desc, scale=scale, head_rows=rows, head_offsets=off)
    else:
        cdesc = cur.make_desc(Kc, Vc, 32)
        Oc, aws = cur.curdkv_attention_out(Q, Kc, Vc, cdesc, scale=scale, head_rows=rows)
    assert cur.curdkv_device_status(aws) == 0
    loss, ref = cur.curdkv_eviction_loss(O, Oc)
    extra = (n - cnt).to(torch.int32).reshape(-1).contiguous()
    if adaptive:
        Oz, _ = cur.curdkv_attention_out(Q, Kc, Vc, desc, scale=scale, head_rows=rows, head_offsets=off,
                                         extra_zero_keys=extra)
    else:
        Oz, _ = cur.curdkv_attention_out(Q, Kc, Vc, cdesc, scale=scale, head_rows=rows, extra_zero_keys=extra)
    loss_z, _ = cur.curdkv_eviction_loss(O, Oz)

    Qf, Kf, Vf = _f64(Q), _f64(K), _f64(V)
    gi, gc, go = idx.cpu().numpy(), cnt.cpu().numpy(), off.cpu().numpy()
    for b in range(B):
        for h in range(H):
            p = b * H + h
            kept = gi[go[p]: go[p] + gc[b, h]] if adaptive else gi[b, h, : gc[b, h]]
            want, want_ref = ev.eviction_loss(Qf[b, h], Kf[b, h], Vf[b, h], kept, scale)
            assert abs(float(loss[b, h]) - want) <= 1e-3 * want_ref, (b, h, float(loss[b, h]), want)
            assert abs(float(ref[b, h]) - want_ref) <= 1e-4 * want_ref
            want_z, _ = ev.eviction_loss(Qf[b, h], Kf[b, h], Vf[b, h], kept, scale, zeroed=True)
            assert abs(float(loss_z[b, h]) - want_z) <= 1e-3 * want_ref
            assert float(loss_z[b, h]) <= ev.lemma1_bound(Vf[b, h], kept)          # Lemma 1
    # keeping every row loses nothing
    same, _ = cur.curdkv_eviction_loss(O, O)
    assert float(same.max()) == 0.0


def test_attention_tiny_and_odd_shapes():
    """One query, one key; 129 queries (two blocks, the second almost empty) over 257 keys."""
    g = torch.Generator(device=DEV).manual_seed(8)
    for m, n in ((1, 1), (129, 257), (128, 128)):
        K = torch.randn((1, 1, n, 128), generator=g, device=DEV).to(torch.bfloat16)
        V = torch.randn((1, 1, n, 128), generator=g, device=DEV).to(torch.bfloat16)
        Q = _queries(1, 1, m, 128, seed=m)
        if n < 128:                       # the tiled loads want at least one full tile of allocation
            Kp = torch.zeros((1, 1, 128, 128), dtype=torch.bfloat16, device=DEV)
            Vp = torch.zeros_like(Kp)
            Kp[:, :, :n], Vp[:, :, :n] = K, V
            desc = cur.make_desc(Kp, Vp, 32, seqlens=torch.tensor([n], dtype=torch.int32, device=DEV))
            O, ws = cur.curdkv_attention_out(Q, Kp, Vp, desc, scale=0.2)
        else:
            desc = cur.make_desc(K, V, 32)
            O, ws = cur.curdkv_attention_out(Q, K, V, desc, scale=0.2)
        assert cur.curdkv_device_status(ws) == 0
        _check_out(O, Q, K, V, np.full((1, 1), n), 0.2, what=f"m={m} n={n}")


def test_attention_running_maximum_moves_every_tile():
    """Logits that grow along the sequence force every tile to raise the running maximum (and each
    warp group to rescale its accumulator); logits that shrink never do.  Both must match the oracle."""
    B, H, n, d, m = 1, 2, 1500, 128, 130
    g = torch.Generator(device=DEV).manual_seed(4)
    ramp = torch.linspace(0.0, 1.0, n, device=DEV).view(1, 1, n, 1)
    for direction in (1.0, -1.0):
        K = torch.randn((B, H, n, d), generator=g, device=DEV) * 0.3
        K[..., 0] += (40.0 * (ramp if direction > 0 else 1.0 - ramp)).squeeze(-1)
        K = K.to(torch.bfloat16)
        V = torch.randn((B, H, n, d), generator=g, device=DEV).to(torch.bfloat16)
        Q = torch.randn((B, H, m, d), generator=g, device=DEV) * 0.3
        Q[..., 0] += 3.0
        Q = Q.to(torch.bfloat16)
        desc = cur.make_desc(K, V, 32)
        O, ws = cur.curdkv_attention_out(Q, K, V, desc, scale=1.0)
        assert cur.curdkv_device_status(ws) == 0
        _check_out(O, Q, K, V, np.full((B, H), n), 1.0, what=f"ramp {direction:+.0f}")


@pytest.mark.parametrize("scale", [-0.3, 0.0])
def test_attention_negative_and_zero_scale(scale):
    """A negative scale turns the row maximum of the logits into a minimum of the raw products
    (the kernel takes the extreme of the unscaled row); scale 0 gives the mean of the value rows.
    Several full tiles and a ragged last one."""
    B, H, n, d, m = 1, 2, 600, 128, 130
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=1, batch=B, n_max=n, kv_heads=H, q_heads=H, data_seed=13)
    K, V, _ = synth.make_kv(w, DEV)
    Q = _queries(B, H, m, d, seed=21)
    desc = cur.make_desc(K, V, 32)
    O, ws = cur.curdkv_attention_out(Q, K, V, desc, scale=scale)
    assert cur.curdkv_device_status(ws) == 0
    _check_out(O, Q, K, V, np.full((B, H), n, dtype=np.int32), scale, what=f"scale={scale}")
    if scale == 0.0:
        mean = _f64(V)[0, 0].mean(axis=0)
        assert np.abs(O.cpu().numpy()[0, 0, 0] - mean).max() <= OUT_TOL * np.abs(mean).max()


def test_attention_rejects_bad_arguments():
    K = torch.zeros((1, 1, 128, 64), dtype=torch.bfloat16, device=DEV)
    Q = torch.zeros((1, 1, 16, 64), dtype=torch.bfloat16, device=DEV)
    desc = cur.make_desc(K, K, 32)
    with pytest.raises(cur.CurdkvError):
        cur.curdkv_attention_out(Q, K, K, desc)
