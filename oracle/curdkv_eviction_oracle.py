"""Eviction loss of a KV selection (Lemma 1 and the reconstruction-loss figure of the paper).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only tests and the benchmark's cpu-baseline
leg may import this module.  Plain numpy in fp64.

For one head with queries Q [m, d], keys K [n, d], values V [n, d] and a kept
index set S:

    O      = softmax(scale * Q K^T) V                      (softmax over the n keys of each row)
    O'     = softmax(scale * Q K_S^T) V_S                  "removed": what a compressed cache computes
    O'_0   = softmax(scale * Q K'^T) V'                    "zeroed": Lemma 1's K', V' keep n rows, the
                                                           evicted ones set to 0 (logit 0, value 0)
    loss   = ||O - O'||_F

Lemma 1 (with the zeroed form): loss <= sqrt(n) ||V - V'||_F + 2 sqrt(n) ||V'||_F.
The paper writes softmax(Q K^T) without a scale; `scale` = 1 reproduces that.
"""
from __future__ import annotations

import numpy as np


def bf16_to_f64(u16):
    return (np.asarray(u16, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def attention_out(Q, K, V, scale=1.0, extra_zero_keys=0):
    """softmax(scale Q K^T) V for fp64 Q [m,d], K [n,d], V [n,d]; `extra_zero_keys` further keys
    with logit 0 and value 0 take part in the softmax (the zeroed rows of Lemma 1)."""
    S = scale * (Q @ K.T)                                   # [m, n]
    top = S.max(axis=1, keepdims=True) if K.shape[0] else np.full((Q.shape[0], 1), -np.inf)
    if extra_zero_keys > 0:
        top = np.maximum(top, 0.0)
    P = np.exp(S - top)
    denom = P.sum(axis=1, keepdims=True) + extra_zero_keys * np.exp(-top)
    return (P @ V) / denom


def eviction_loss(Q, K, V, kept, scale=1.0, zeroed=False):
    """(||O - O'||_F, ||O||_F) for the kept row indices `kept` of K, V."""
    kept = np.asarray(kept, dtype=np.int64)
    O = attention_out(Q, K, V, scale)
    Oc = attention_out(Q, K[kept], V[kept], scale, extra_zero_keys=(K.shape[0] - len(kept)) if zeroed else 0)
    return float(np.linalg.norm(O - Oc)), float(np.linalg.norm(O))


def lemma1_bound(V, kept):
    """sqrt(n) ||V - V'||_F + 2 sqrt(n) ||V'||_F with V' = V with the evicted rows zeroed."""
    n = V.shape[0]
    Vp = np.zeros_like(V)
    Vp[np.asarray(kept, dtype=np.int64)] = V[np.asarray(kept, dtype=np.int64)]
    return float(np.sqrt(n) * np.linalg.norm(V - Vp) + 2 * np.sqrt(n) * np.linalg.norm(Vp))
