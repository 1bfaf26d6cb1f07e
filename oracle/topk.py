"""Oracle: beam x codebook top-k and the beam-state update.  Test infrastructure.

Section 3.1 / 3.3: per request, the K = M_{t+1} highest-scoring candidates of
the M_t * |V| scored children form the next beam; the selected children's
parent rows, tokens, scores and trie node ids become the next beam state.

Readings where the paper is silent: candidates are ordered by value descending
and, for equal values, by ascending flat index m * V + v; -0.0 equals +0.0;
-inf takes part like any other value, and a selected -inf yields a dead beam
(node -1).  Output row i is the i-th candidate of that order.
"""
from __future__ import annotations

import numpy as np

U64 = np.uint64


def beam_topk(cand: np.ndarray, K: int, V: int):
    """cand fp32 [B, N] -> (score f32, flat i32, parent i32, token i32), each [B, K]."""
    cand = np.asarray(cand, dtype=np.float32)
    B, N = cand.shape
    assert K > 0
    assert not np.isnan(cand).any(), "NaN candidates violate the precondition"
    # A beam wider than the candidate set (Section 3.3: the fixed schedule asks for 1024 beams where at
    # most |V| = 512 prefixes exist): every candidate in order, then dead entries (-inf on candidate 0).
    score = np.full((B, K), -np.inf, dtype=np.float32)
    flat = np.zeros((B, K), dtype=np.int32)
    k = min(K, N)
    for b in range(B):
        row = cand[b] + np.float32(0.0)               # -0.0 -> +0.0
        order = np.argsort(-row, kind="stable")       # stable: ties keep index order
        flat[b, :k] = order[:k]
        score[b, :k] = cand[b, order[:k]]
    return score, flat, (flat // V).astype(np.int32), (flat % V).astype(np.int32)


def update_beam_state(trie, parent, token, score, prev_node, prev_key, prefix_len, M_prev):
    """New beam state after top-k (Section 3.3 "rearrangement", Section 4.4).

    parent/token/score [B, K] from `beam_topk`; prev_node/prev_key [B * M_prev].
    Returns (node int32 [B*K], key uint64 [B*K]).  No KV bytes move: the parent
    array itself is what the next self-attention follows.
    """
    B, K = parent.shape
    node = np.full(B * K, -1, dtype=np.int32)
    key = np.zeros(B * K, dtype=U64)
    for b in range(B):
        for i in range(K):
            src = b * M_prev + int(parent[b, i])
            key[b * K + i] = U64(prev_key[src]) | (U64(int(token[b, i]) + 1) << U64(16 * prefix_len))
            if np.isneginf(score[b, i]) or prev_node[src] < 0:
                continue
            node[b * K + i] = trie.child(int(prev_node[src]), int(token[b, i]))
    return node, key
