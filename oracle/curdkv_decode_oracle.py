"""Generation-phase use of CurDKV, step by step (plain numpy over the fp64 C oracle).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only tests and the benchmark's cpu-baseline
leg may import this module.

Sec. 3.2 states that the method applies while tokens are generated as well as at
prefill, without spelling the procedure out.  The reading restated here: a cache
holds, per (sequence, KV head), rows of K and V with their original token
positions and their unnormalised combined scores l^KV_j = l^K_j * l^V_j
(Alg. 1 (sketch, row norms, product); a row's score depends only on that row and on G).  Newly
generated rows are appended with their scores.  A compression step applies
Alg. 1 (normalisation, selection, gather) to the rows held at that moment: normalise over them, keep the
sinks (positions < s), the most recent `window` positions and the best-scoring
rest up to the budget k, in ascending position order.

Pinned (parity pinned): after any schedule of appends and compressions the kept
positions equal those of ONE application of Alg. 1 to the whole history with the
same k, s and window (top-k of a union equals top-k of the union of a top-k with
the rest; forced tokens only ever turn into ordinary candidates).
"""
from __future__ import annotations

import numpy as np

from oracle import curdkv_oracle as orc


def raw_scores(K, V, G):
    """l^K_j * l^V_j in fp64 for bf16 bit patterns K, V [B,H,n,d] (Alg. 1 (sketch, row norms, product))."""
    _, _, lK, lV = orc.score(K, V, G, return_factors=True)
    return lK * lV


class CacheOracle:
    """Cache of one layer: per sequence b a common row count, per (b, h) positions, scores, rows."""

    def __init__(self, B, H, d):
        self.B, self.H, self.d = B, H, d
        self.pos = [[np.zeros((0,), np.int64) for _ in range(H)] for _ in range(B)]
        self.raw = [[np.zeros((0,), np.float64) for _ in range(H)] for _ in range(B)]
        self.K = [[np.zeros((0, d), np.uint16) for _ in range(H)] for _ in range(B)]
        self.V = [[np.zeros((0, d), np.uint16) for _ in range(H)] for _ in range(B)]
        self.total = np.zeros((B,), np.int64)

    def append(self, K_new, V_new, G, t_new=None):
        """K_new, V_new: uint16 [B,H,t,d]; t_new[b] <= t rows of sequence b are real."""
        B, H, t, _ = K_new.shape
        t_new = np.full((B,), t, np.int64) if t_new is None else np.asarray(t_new, np.int64)
        raw = raw_scores(K_new, V_new, G)
        for b in range(B):
            tb = int(t_new[b])
            for h in range(H):
                self.pos[b][h] = np.concatenate([self.pos[b][h], self.total[b] + np.arange(tb)])
                self.raw[b][h] = np.concatenate([self.raw[b][h], raw[b, h, :tb]])
                self.K[b][h] = np.concatenate([self.K[b][h], K_new[b, h, :tb]])
                self.V[b][h] = np.concatenate([self.V[b][h], V_new[b, h, :tb]])
            self.total[b] += tb

    def compress(self, budget, num_sink, window):
        """Alg. 1 (normalisation, selection, gather) on the held rows of every (b, h)."""
        for b in range(self.B):
            for h in range(self.H):
                raw = self.raw[b][h]
                n = raw.shape[0]
                if n == 0:
                    continue
                S = raw.sum()
                norm = raw / S if S > 0 else np.zeros_like(raw)          # normalise
                idx, cnt = orc.select_fixed(norm[None, None, :], budget, num_sink, window)  # sinks, top-k, union
                keep = idx[0, 0, : cnt[0, 0]]
                self.pos[b][h] = self.pos[b][h][keep]                     # gather (+ bookkeeping)
                self.raw[b][h] = raw[keep]
                self.K[b][h] = self.K[b][h][keep]
                self.V[b][h] = self.V[b][h][keep]

    def counts(self):
        return np.array([[len(self.pos[b][h]) for h in range(self.H)] for b in range(self.B)])
