"""k-way partitioned matcher rows.  TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

Section 4.2 ("k-way partition"), Section 4.3 (last paragraph) and Section 4.4 (last paragraph):
instead of one OR-union row per trie node, the SIDs below a node are split into up to k groups and
one union row is stored per group; a prefix is kept if ANY group matches every attribute (bitmask
containment) and any request location (Bloom containment).  Static k-way fixes k per decode
position; dynamic k-way raises k per node until the fill rate of its rows reaches a target or k_max.

Readings taken here (the paper gives the rule, not the details):
  * a partition carries a pair (bitmask row, Bloom row) and both tests are made on the same pair;
  * fill rate of a pair = set bits of the two rows / their total width;
  * construction is greedy in SID order: a SID joins the group whose pair has the smallest fill after
    OR-ing the SID's rows in (ties: lowest group number); groups that stay empty are not stored;
  * the fill rate of a node is that of its fullest group; dynamic k-way takes the smallest k in
    1..min(k_max, #SIDs below) whose node fill is <= the target, else that upper bound;
  * storage is the jagged form (per-entry offsets into flat id arrays); the fixed-width layout of
    static k-way is the special case of equal row lengths.

PIN STATUS: pinned by tests/test_oracle_kway.py (k = 1 equals the unpartitioned index; brute-force
ad-level eligibility is never lost; partition pass implies union pass; one group per SID is exact at
SID level; the Section 4.2 worked example is filtered once its two ads sit in different groups).
"""
from __future__ import annotations

import numpy as np

from .matchers import bitmask_match, bloom_any

U64 = np.uint64


def _popcount_rows(rows: np.ndarray) -> np.ndarray:
    """Set bits per row of a uint64 [n, W] array."""
    b = np.ascontiguousarray(rows).view(np.uint8).reshape(rows.shape[0], -1)
    return np.unpackbits(b, axis=1).sum(axis=1).astype(np.int64)


def sid_rows(n_sids: int, ad_sid: np.ndarray, ad_bitmask: np.ndarray, ad_bloom: np.ndarray):
    """Rows of a SID = OR of the rows of its ads (the union rule of Section 4.2 applied at the leaf)."""
    order = np.argsort(ad_sid, kind="stable")
    starts = np.searchsorted(ad_sid[order], np.arange(n_sids))
    return (np.bitwise_or.reduceat(ad_bitmask[order], starts, axis=0),
            np.bitwise_or.reduceat(ad_bloom[order], starts, axis=0))


def greedy_groups(bm: np.ndarray, bl: np.ndarray, k: int):
    """Split the SIDs (rows of bm / bl, in order) into at most k groups; returns the groups' union
    rows (bitmask [g, W_bm], Bloom [g, W_bl]) with g <= k non-empty groups, in group order."""
    n = bm.shape[0]
    g_bm = np.zeros((k, bm.shape[1]), dtype=U64)
    g_bl = np.zeros((k, bl.shape[1]), dtype=U64)
    used = np.zeros(k, dtype=bool)
    for i in range(n):
        after = _popcount_rows(g_bm | bm[i]) + _popcount_rows(g_bl | bl[i])
        p = int(np.argmin(after))                       # first minimum = lowest group number
        g_bm[p] |= bm[i]
        g_bl[p] |= bl[i]
        used[p] = True
    return g_bm[used], g_bl[used]


def node_fill(g_bm: np.ndarray, g_bl: np.ndarray) -> float:
    bits = 64 * (g_bm.shape[1] + g_bl.shape[1])
    return float((_popcount_rows(g_bm) + _popcount_rows(g_bl)).max()) / bits


class KWayMatcherIndex:
    """part_offsets [E + 1]; bitmask_index / bloom_index [P] into tables of unique rows.

    policy: ("static", k_level) with k_level[l] the k of child entries that lead to nodes of level l
    (l = 1..L), or ("dynamic", fill_target, k_max).
    """

    def __init__(self, trie, sids: np.ndarray, ad_sid, ad_bitmask, ad_bloom, policy):
        L = trie.sid_length
        leaf_bm, leaf_bl = sid_rows(sids.shape[0], ad_sid, ad_bitmask, ad_bloom)
        E = trie.num_nodes - 1
        offsets = np.zeros(E + 1, dtype=np.int64)
        self.part_k = np.zeros(E, dtype=np.int32)                 # the k each entry was built with
        rows_bm, rows_bl = [], []
        for l in range(1, L + 1):
            change = np.any(sids[1:, :l] != sids[:-1, :l], axis=1)
            first = np.concatenate([[0], np.nonzero(change)[0] + 1, [sids.shape[0]]])
            base = int(trie.level_start[l])
            for i in range(first.shape[0] - 1):
                lo, hi = int(first[i]), int(first[i + 1])          # the SIDs below node base + i
                bm, bl = leaf_bm[lo:hi], leaf_bl[lo:hi]
                if policy[0] == "static":
                    k = max(1, min(int(policy[1][l]), hi - lo))
                    g_bm, g_bl = greedy_groups(bm, bl, k)
                else:
                    target, k_max = float(policy[1]), int(policy[2])
                    k_top = max(1, min(k_max, hi - lo))
                    for k in range(1, k_top + 1):
                        g_bm, g_bl = greedy_groups(bm, bl, k)
                        if node_fill(g_bm, g_bl) <= target:
                            break
                entry = base + i - 1                                # entry j leads to node j + 1
                self.part_k[entry] = k
                offsets[entry + 1] = g_bm.shape[0]
                rows_bm.append((entry, g_bm))
                rows_bl.append((entry, g_bl))
        self.part_offsets = np.cumsum(offsets).astype(np.int32)
        rows_bm.sort(key=lambda t: t[0])
        rows_bl.sort(key=lambda t: t[0])
        all_bm = np.concatenate([r for _, r in rows_bm], axis=0)
        all_bl = np.concatenate([r for _, r in rows_bl], axis=0)
        self.part_bitmask_rows, self.part_bloom_rows = all_bm, all_bl      # before deduplication
        self.bitmask_table, idx = np.unique(all_bm, axis=0, return_inverse=True)
        self.bitmask_index = idx.reshape(-1).astype(np.int32)
        self.bloom_table, idx = np.unique(all_bl, axis=0, return_inverse=True)
        self.bloom_index = idx.reshape(-1).astype(np.int32)

    def entry_passes(self, entry: int, user_bitmask: np.ndarray, user_blooms: np.ndarray) -> bool:
        for p in range(int(self.part_offsets[entry]), int(self.part_offsets[entry + 1])):
            if (bitmask_match(self.bitmask_table[self.bitmask_index[p]], user_bitmask)
                    and bloom_any(self.bloom_table[self.bloom_index[p]], user_blooms)):
                return True
        return False


class KWayRowsMatcher:
    """TM for `oracle.gtm.gtm_mask`: kept if ANY group of the child's node passes both tests."""

    def __init__(self, trie, index: KWayMatcherIndex, user_bitmask: np.ndarray, user_blooms: np.ndarray):
        self.trie, self.index = trie, index
        self.user_bitmask, self.user_blooms = user_bitmask, user_blooms

    def match(self, request, row_key, prefix_len, tokens, child_nodes):
        out = np.zeros(tokens.shape[0], dtype=bool)
        for i, child in enumerate(child_nodes):
            out[i] = self.index.entry_passes(int(child) - 1, self.user_bitmask[request], self.user_blooms[request])
        return out
