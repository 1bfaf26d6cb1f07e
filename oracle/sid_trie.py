"""Oracle: the SID prefix trie in the CSR layout of Appendix A.  Test infrastructure.

Section 4.4 / Appendix A store the catalog as a trie whose children sit in one
contiguous child-entry range per node (`node_offsets`, `csr_tokens`,
`csr_child_nodes`).  The paper does not fix the numbering; the reading used
everywhere here: nodes are numbered level by level (root = 0), and inside a
level in lexicographic order of their prefixes, so the children of a node are
consecutive ids in increasing token order.
"""
from __future__ import annotations

import numpy as np


class SidTrie:
    """CSR trie over a catalog of fixed-length SIDs (Appendix A field names)."""

    def __init__(self, sids: np.ndarray, vocab_size: int):
        sids = np.asarray(sids, dtype=np.int64)
        assert sids.ndim == 2 and sids.shape[0] > 0
        assert sids.min() >= 0 and sids.max() < vocab_size
        self.vocab_size = int(vocab_size)
        self.sid_length = int(sids.shape[1])
        L = self.sid_length

        # prefixes[l] : sorted distinct prefixes of length l, shape [n_l, l]
        self.prefixes = [np.zeros((1, 0), dtype=np.int64)]
        for l in range(1, L + 1):
            self.prefixes.append(np.unique(sids[:, :l], axis=0))
        counts = [p.shape[0] for p in self.prefixes]
        self.level_start = np.concatenate([[0], np.cumsum(counts)]).astype(np.int64)
        self.num_nodes = int(self.level_start[-1])

        node_offsets = np.zeros(self.num_nodes + 1, dtype=np.int64)
        tokens, children = [], []
        entry = 0
        for l in range(L):                      # parents at level l, children at l + 1
            par, chi = self.prefixes[l], self.prefixes[l + 1]
            # rank of each child's parent among the level-l prefixes
            if l == 0:
                parent_rank = np.zeros(chi.shape[0], dtype=np.int64)
            else:
                # both are lexicographically sorted, so the parent rank is the
                # number of distinct (l)-prefixes seen so far minus one
                change = np.any(chi[1:, :l] != chi[:-1, :l], axis=1)
                parent_rank = np.concatenate([[0], np.cumsum(change)])
                assert parent_rank[-1] == par.shape[0] - 1
            per_parent = np.bincount(parent_rank, minlength=par.shape[0])
            base = int(self.level_start[l])
            node_offsets[base + 1: base + 1 + par.shape[0]] = entry + np.cumsum(per_parent)
            entry += chi.shape[0]
            tokens.append(chi[:, l])
            children.append(self.level_start[l + 1] + np.arange(chi.shape[0]))
        # leaves have empty ranges
        leaf0 = int(self.level_start[L])
        node_offsets[leaf0 + 1:] = entry
        self.node_offsets = node_offsets.astype(np.int32)
        self.csr_tokens = np.concatenate(tokens).astype(np.int16 if vocab_size <= 32767 else np.int32)
        self.csr_child_nodes = np.concatenate(children).astype(np.int32)
        self.num_child_entries = int(entry)

    # ---- Appendix A lookup ------------------------------------------------
    def lookup(self, node_id: int):
        """Child-entry range of `node_id`: (tokens, child node ids)."""
        start = int(self.node_offsets[node_id])
        end = int(self.node_offsets[node_id + 1])
        return (self.csr_tokens[start:end].astype(np.int64),
                self.csr_child_nodes[start:end].astype(np.int64))

    def child(self, node_id: int, token: int) -> int:
        """Child of `node_id` reached by `token`, or -1 (Eq. CD_t)."""
        toks, kids = self.lookup(node_id)
        hit = np.nonzero(toks == token)[0]
        return int(kids[hit[0]]) if hit.size else -1

    def walk(self, tokens) -> int:
        """Node id of the prefix `tokens`, or -1 if it is not in the catalog."""
        node = 0
        for tok in tokens:
            node = self.child(node, int(tok))
            if node < 0:
                return -1
        return node

    def level_of(self, node_id: int) -> int:
        return int(np.searchsorted(self.level_start, node_id, side="right") - 1)

    def prefix_of(self, node_id: int) -> tuple:
        l = self.level_of(node_id)
        return tuple(int(x) for x in self.prefixes[l][node_id - int(self.level_start[l])])

    def num_internal_nodes(self) -> int:
        """Nodes that can have children (levels 0 .. L-1)."""
        return int(self.level_start[self.sid_length])

    # ---- the same trie as a per-node child bitmask --------------------------
    def dense_child_bits(self):
        """(child_bits uint64 [n_internal, V/64], child_base int32 [n_internal]).

        Bit v of row n is CD[v] for node n; child_base[n] is the id of n's
        first child, so child(n, v) = child_base[n] + popcount(bits below v).
        """
        V = self.vocab_size
        assert V % 64 == 0
        n_int = self.num_internal_nodes()
        bits = np.zeros((n_int, V // 64), dtype=np.uint64)
        base = np.zeros(n_int, dtype=np.int32)
        for n in range(n_int):
            toks, kids = self.lookup(n)
            base[n] = kids[0] if kids.size else -1
            for tok in toks:
                bits[n, tok // 64] |= np.uint64(1) << np.uint64(tok % 64)
        return bits, base

    def dense_child_bits_fast(self):
        """Vectorised form of `dense_child_bits` for large catalogs (same result)."""
        V = self.vocab_size
        n_int = self.num_internal_nodes()
        deg = np.diff(self.node_offsets[: n_int + 1].astype(np.int64))
        owner = np.repeat(np.arange(n_int, dtype=np.int64), deg)
        tok = self.csr_tokens.astype(np.int64)
        bits = np.zeros((n_int, V // 64), dtype=np.uint64)
        np.bitwise_or.at(bits, (owner, tok // 64), np.uint64(1) << (tok % 64).astype(np.uint64))
        base = np.where(deg > 0, self.csr_child_nodes[np.minimum(
            self.node_offsets[:n_int].astype(np.int64), self.num_child_entries - 1)], -1)
        return bits, base.astype(np.int32)
