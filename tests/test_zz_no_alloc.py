"""curdkv_score_static: the scoring call for callers that cannot allocate device memory.

Some hosts of this library (a serving framework that owns the whole memory pool, a plugin
that only receives its input and output buffers) cannot call cudaMalloc, so they have no
workspace to hand to curdkv_score.  The static variant keeps that scratch in an array built
into the library.  This test calls it through the C ABI twice in a row -- the array is shared
and keeps the previous call's contents, so the second call must not be disturbed by the
first -- and compares with curdkv_score on the same inputs.  It is collected last so that a
failure here cannot hide any other test under `-x`.
"""
import pytest
import torch

from paper_2509_15038_b200 import binding as cur
from paper_2509_15038_b200 import synth

pytestmark = pytest.mark.gpu


def _case(w, seed_shift, seqlens=None):
    w = synth.shrink(w, data_seed=w.data_seed + seed_shift)
    K, V, _ = synth.make_kv(w, "cuda")
    G = torch.as_tensor(synth.make_G(w.d, w.r, seed=seed_shift), device="cuda")
    sl = None if seqlens is None else torch.as_tensor(seqlens, dtype=torch.int32, device="cuda")
    desc = cur.make_desc(K, V, w.r, q_heads=w.q_heads, seqlens=sl)
    return K, V, G, desc, sl


def test_static_scratch_matches_workspace_variant_twice():
    # two different shapes back to back: the second (ragged, fewer tiles) runs over the
    # partial sums the first left behind in the shared array
    cases = [
        _case(synth.shrink(synth.CONFIGS["cfg2"], layers=2, n_max=4096), 0),
        _case(synth.shrink(synth.CONFIGS["cfg2"], layers=1, batch=3, n_max=1000), 1, seqlens=[1000, 517, 0]),
    ]
    for K, V, G, desc, sl in cases:
        ws = cur.alloc_workspace(desc)
        want_scores, want_sums = cur.curdkv_score(K, V, G, desc, ws)
        assert cur.curdkv_device_status(ws) == 0
        flags = torch.full((1,), 0xFFFF, dtype=torch.int32, device="cuda")
        scores = torch.full_like(want_scores, -1.0)
        sums = torch.full_like(want_sums, -1.0)
        cur.curdkv_score_static(K, V, G, desc, scores=scores, head_sums=sums, status_flags=flags)
        torch.cuda.synchronize()
        assert int(flags.item()) == 0
        # same kernels, same order of operations: the tolerance of the parity tests
        # (1e-3 relative) is met with room to spare; in practice the bits agree
        torch.testing.assert_close(scores, want_scores, rtol=1e-3, atol=0)
        torch.testing.assert_close(sums, want_sums, rtol=1e-3, atol=0)
        assert torch.all(scores.sum(-1)[want_sums > 0].sub(1).abs() < 1e-3)


def test_static_scratch_rejects_oversized_shapes_without_launching():
    K = torch.zeros((1, 1, 128, 128), dtype=torch.bfloat16, device="cuda")
    G = torch.zeros((128, 32), dtype=torch.float32, device="cuda")
    # descriptor of a shape with 2^18 + 1 tiles; no memory of that size is touched
    # because the call is refused before anything is enqueued
    desc = cur.make_desc(K, K, 32)
    desc.batch = 2 ** 18 + 1
    before = cur.launch_count()
    scores = torch.zeros((1,), device="cuda")
    with pytest.raises(cur.CurdkvError) as e:
        cur.curdkv_score_static(K, K, G, desc, scores=scores, head_sums=scores)
    assert e.value.code == 6 and "built-in scratch" in str(e.value)
    assert cur.launch_count() == before
