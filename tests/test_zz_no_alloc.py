"""curdkv_score_static: the scoring call for callers that cannot allocate device memory.

Some hosts of this library (a serving framework that owns the whole memory pool, a plugin
that only receives its input and output buffers) cannot call cudaMalloc, so they have no
workspace to hand to curdkv_score.  The static variant keeps that scratch in an array built
into the library.  This test calls it through the C ABI twice in a row -- the array is shared
and keeps the previous call's contents, so the second call must not be disturbed by the
first -- and compares with curdkv_score on the same inputs (the same kernels in the same
order: the bits must agree) and with the fp64 oracle.  It is collected last so that a failure
here cannot hide any other test under `-x`.
"""
import numpy as np
import pytest
import torch

from oracle import curdkv_oracle as orc
from paper_2509_15038_b200 import binding as cur
from paper_2509_15038_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def _case(w, seed_shift, seqlens=None):
    w = synth.shrink(w, data_seed=w.data_seed + seed_shift)
    K, V, _ = synth.make_kv(w, "cuda")
    G = torch.as_tensor(synth.make_G(w.d, w.r, seed=seed_shift), device="cuda")
    sl = None if seqlens is None else torch.as_tensor(seqlens, dtype=torch.int32, device="cuda")
    desc = cur.make_desc(K, V, w.r, q_heads=w.q_heads, seqlens=sl)
    return K, V, G, desc, (sl, seqlens)         # desc points at sl: keep it alive


def test_static_scratch_matches_workspace_variant_twice():
    # two different shapes back to back: the second (ragged, fewer tiles) runs over the
    # partial sums the first left behind in the shared array
    cases = [
        _case(synth.shrink(synth.CONFIGS["cfg2"], layers=2, n_max=4096), 0),
        _case(synth.shrink(synth.CONFIGS["cfg2"], layers=1, batch=3, n_max=1000), 1, seqlens=[1000, 517, 0]),
    ]
    for K, V, G, desc, (_, lens) in cases:
        ws = cur.alloc_workspace(desc)
        want_scores, want_sums = cur.curdkv_score(K, V, G, desc, ws)
        assert cur.curdkv_device_status(ws) == 0
        flags = torch.full((1,), 0xFFFF, dtype=torch.int32, device="cuda")
        scores = torch.full_like(want_scores, -1.0)
        sums = torch.full_like(want_sums, -1.0)
        cur.curdkv_score_static(K, V, G, desc, scores=scores, head_sums=sums, status_flags=flags)
        torch.cuda.synchronize()
        assert int(flags.item()) == 0
        assert torch.equal(scores, want_scores) and torch.equal(sums, want_sums)
        # and against the oracle, at the tolerance of the parity tests
        rs, rS = orc.score(synth.to_u16(K), synth.to_u16(V), G.cpu().numpy(),
                           seqlens=None if lens is None else np.asarray(lens, dtype=np.int32))
        pu.assert_scores_close(scores.cpu().numpy(), rs, "static scratch")
        np.testing.assert_allclose(sums.cpu().numpy(), rS, rtol=1e-4)


def test_static_call_leaves_device_memory_as_it_is():
    """After a first call (which looks up the array's address), further calls change neither the
    free device memory nor torch's own allocation count: nothing is allocated on any route."""
    K, V, G, desc, _ = _case(synth.shrink(synth.CONFIGS["cfg2"], layers=1, n_max=2048), 2)
    scores = torch.empty((desc.batch, desc.kv_heads, desc.n_max), dtype=torch.float32, device="cuda")
    sums = torch.empty((desc.batch, desc.kv_heads), dtype=torch.float32, device="cuda")
    cur.curdkv_score_static(K, V, G, desc, scores=scores, head_sums=sums)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    allocs0 = torch.cuda.memory_stats()["allocation.all.allocated"]
    for _ in range(3):
        cur.curdkv_score_static(K, V, G, desc, scores=scores, head_sums=sums)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert torch.cuda.memory_stats()["allocation.all.allocated"] == allocs0


def test_static_scratch_rejects_oversized_and_whitened_shapes_without_launching():
    K = torch.zeros((1, 1, 128, 128), dtype=torch.bfloat16, device="cuda")
    G = torch.zeros((128, 32), dtype=torch.float32, device="cuda")
    # descriptor of a shape with 2^18 + 1 tiles; no memory of that size is touched
    # because the call is refused before anything is enqueued
    desc = cur.make_desc(K, K, 32)
    desc.batch = 2 ** 18 + 1
    before = cur.launch_count()
    scores = torch.zeros((128,), device="cuda")
    with pytest.raises(cur.CurdkvError) as e:
        cur.curdkv_score_static(K, K, G, desc, scores=scores, head_sums=scores)
    assert e.value.code == 6 and "built-in scratch" in str(e.value)
    # the whitened mode needs Gram matrices in its scratch: not offered by the static call,
    # however small the shape
    white = cur.make_desc(K, K, 32, whiten=1, ridge=1e-4)
    with pytest.raises(cur.CurdkvError) as e:
        cur.curdkv_score_static(K, K, G, white, scores=scores, head_sums=scores)
    assert e.value.code == 2
    assert cur.launch_count() == before
