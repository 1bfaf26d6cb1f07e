"""Oracle: CD + GTM masking of next-token log-probabilities.  Test infrastructure.

Section 4.1: CD_t[v] = 1[v in children(p)], TM_t[v] = match(u, p || v), and a
candidate keeps its log-probability only when CD_t[v] * TM_t[v] = 1, otherwise
it becomes -inf.  Section 3.1: the score of a surviving child is the prefix's
accumulated log-probability plus the token's log-probability.

Readings where the paper is silent: the mask is applied to log-probabilities
that were normalised over the whole vocabulary (no renormalisation afterwards);
the score update is one fp32 round-to-nearest add; a beam whose node id is -1
is dead and has no allowed child.
"""
from __future__ import annotations

import numpy as np

from .matchers import PrefixBloom

U64 = np.uint64


class NoMatcher:
    """TM = 1 everywhere: constrained decoding only."""

    def match(self, request, row_key, prefix_len, tokens, child_nodes):
        return np.ones(tokens.shape[0], dtype=bool)


class NodeBitmaskMatcher:
    """Per-request eligibility bit for every trie node (bool [B, num_nodes])."""

    def __init__(self, node_marks: np.ndarray):
        self.node_marks = np.asarray(node_marks, dtype=bool)

    def match(self, request, row_key, prefix_len, tokens, child_nodes):
        return self.node_marks[request, child_nodes]


class PrefixBloomMatcher:
    """Per-request Bloom filter over prefix keys."""

    def __init__(self, blooms):
        self.blooms = list(blooms)
        assert all(isinstance(b, PrefixBloom) for b in self.blooms)

    def match(self, request, row_key, prefix_len, tokens, child_nodes):
        child_keys = U64(row_key) | ((tokens + 1).astype(U64) << U64(16 * prefix_len))
        return self.blooms[request].contains(child_keys)


def gtm_mask(logp, beam_score, beam_node, beam_key, prefix_len, trie, matcher, B, M):
    """Mask and score one step's candidates.

    logp        fp32 [B*M, V]   next-token log-probabilities
    beam_score  fp32 [B*M]      accumulated log-probability of each prefix
    beam_node   int  [B*M]      trie node id of each prefix, -1 = dead beam
    beam_key    u64  [B*M]      prefix key (used by the Bloom matcher)
    prefix_len  int             number of tokens already decoded (= step index t)

    Returns (cand fp32 [B*M, V], allow bool [B*M, V], child_node int32 [B*M, V]).
    """
    logp = np.asarray(logp, dtype=np.float32)
    R, V = logp.shape
    assert R == B * M
    cand = np.full((R, V), -np.inf, dtype=np.float32)
    allow = np.zeros((R, V), dtype=bool)
    child_node = np.full((R, V), -1, dtype=np.int32)
    for r in range(R):
        node = int(beam_node[r])
        if node < 0:
            continue
        tokens, kids = trie.lookup(node)                 # CD: the node's children
        if tokens.size == 0:
            continue
        ok = matcher.match(r // M, beam_key[r], prefix_len, tokens, kids)   # TM
        tokens, kids = tokens[ok], kids[ok]
        allow[r, tokens] = True
        child_node[r, tokens] = kids
        cand[r, tokens] = np.float32(beam_score[r]) + logp[r, tokens]       # fp32 add
    return cand, allow, child_node


def pack_allow_bits(allow: np.ndarray) -> np.ndarray:
    """bool [R, V] -> uint64 [R, V/64]; token v is bit (v & 63) of word (v >> 6)."""
    R, V = allow.shape
    assert V % 64 == 0
    weights = U64(1) << np.arange(64, dtype=U64)
    return (allow.reshape(R, V // 64, 64).astype(U64) * weights).sum(axis=2, dtype=U64)
