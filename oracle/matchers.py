"""Oracle: targeting matchers TM_t[v] = match(u, p || v).  Test infrastructure.

Two families, both instances of the Section 4.1 indicator:

* The paper's per-node rows (Sections 4.2, 4.3): every trie node stores the OR
  of its ads' attribute bitmasks / Bloom rows; a request carries one attribute
  bitmask and a list of location Bloom rows.
* Per-request structures over SID prefixes (the forms the benchmark
  configurations name): an eligibility bit per trie node, or a Bloom filter of
  prefix keys.  "Eligible prefix" follows Section 4.1: a prefix whose subtree
  holds at least one eligible SID.

The hash of the prefix Bloom filter is not given by the paper; the reading
used: key = sum_i (token_i + 1) << 16 i, mixed by the splitmix64 finaliser,
double hashing with h1 = low word, h2 = high word | 1, probe_i = (h1 + i h2)
mod 2^32 mod m.
"""
from __future__ import annotations

import numpy as np

U64 = np.uint64


# ---------------------------------------------------------------------------
# Paper forms (Sections 4.2 and 4.3)
# ---------------------------------------------------------------------------
def union_rows(rows: np.ndarray) -> np.ndarray:
    """Stored matcher of a node: OR over the rows of the ads below it."""
    rows = np.asarray(rows, dtype=U64)
    return np.bitwise_or.reduce(rows, axis=0)


def bitmask_match(node_bitmask: np.ndarray, user_bitmask: np.ndarray) -> bool:
    """Section 4.2 packed test: every user attribute bit is present in the node row."""
    node_bitmask = np.asarray(node_bitmask, dtype=U64)
    user_bitmask = np.asarray(user_bitmask, dtype=U64)
    return bool(np.all((node_bitmask & user_bitmask) == user_bitmask))


def bloom_contains(stored: np.ndarray, location_row: np.ndarray) -> bool:
    """Section 4.3 containment: (bloom(l) AND B) == bloom(l)."""
    stored = np.asarray(stored, dtype=U64)
    location_row = np.asarray(location_row, dtype=U64)
    return bool(np.all((location_row & stored) == location_row))


def bloom_any(stored: np.ndarray, user_location_rows) -> bool:
    """ANY-of-many location predicate; an empty location list matches nothing."""
    return any(bloom_contains(stored, q) for q in user_location_rows)


def paper_lookup(trie, bitmask_index, bloom_index, bitmask_table, bloom_table,
                 node_id: int, user_bitmask, user_blooms):
    """The index lookup of Appendix A for one node and one request: the (token, child node) pairs the
    request may extend the node's prefix with.

    Stated as a filter over the node's child entries (the CSR range of the node): an entry survives iff its
    attribute row contains the request's attribute row (Section 4.2) and its Bloom row contains at least one
    of the request's location rows (Section 4.3; none at all if the request has no location)."""
    entries = np.arange(int(trie.node_offsets[node_id]), int(trie.node_offsets[node_id + 1]))
    if entries.size == 0:
        return []
    attr_rows = np.asarray(bitmask_table)[np.asarray(bitmask_index)[entries]]           # [n, W_bm]
    bloom_rows = np.asarray(bloom_table)[np.asarray(bloom_index)[entries]]              # [n, W_bl]
    want = np.asarray(user_bitmask, dtype=U64)
    attr_ok = ((attr_rows & want[None, :]) == want[None, :]).all(axis=1)
    locs = np.asarray(user_blooms, dtype=U64).reshape(-1, bloom_rows.shape[1])          # [N_loc, W_bl]
    loc_ok = ((bloom_rows[:, None, :] & locs[None, :, :]) == locs[None, :, :]).all(axis=2).any(axis=1)
    keep = entries[attr_ok & loc_ok]
    return [(int(trie.csr_tokens[j]), int(trie.csr_child_nodes[j])) for j in keep]


# ---------------------------------------------------------------------------
# Per-request forms over prefixes
# ---------------------------------------------------------------------------
def node_eligibility(trie, sids: np.ndarray, eligible: np.ndarray) -> np.ndarray:
    """bool [num_nodes]: node n is set iff some eligible SID has n's prefix.

    Written as the definition: walk every eligible SID from the root and mark
    each node on its path.
    """
    marks = np.zeros(trie.num_nodes, dtype=bool)
    marks[0] = bool(np.any(eligible))
    L = trie.sid_length
    for l in range(1, L + 1):
        pref = trie.prefixes[l]
        sel = np.unique(np.asarray(sids)[np.asarray(eligible, dtype=bool)][:, :l], axis=0)
        if sel.shape[0] == 0:
            continue
        # rank of each selected prefix among the level's sorted prefixes
        rank = _rows_rank(pref, sel)
        marks[int(trie.level_start[l]) + rank] = True
    return marks


def _rows_rank(sorted_rows: np.ndarray, query_rows: np.ndarray) -> np.ndarray:
    """Index of each query row inside a lexicographically sorted row set."""
    def pack(a):
        k = np.zeros(a.shape[0], dtype=np.uint64)
        for j in range(a.shape[1]):
            k = (k << U64(16)) | a[:, j].astype(U64)
        return k
    ks, kq = pack(sorted_rows), pack(query_rows)
    idx = np.searchsorted(ks, kq)
    assert np.all(ks[idx] == kq)
    return idx


def pack_node_bits(marks: np.ndarray) -> np.ndarray:
    """bool [n] -> uint64 words, bit (n & 63) of word (n >> 6)."""
    n = marks.shape[0]
    words = (n + 63) // 64
    padded = np.zeros(words * 64, dtype=bool)
    padded[:n] = marks
    weights = (U64(1) << np.arange(64, dtype=U64))
    return (padded.reshape(words, 64).astype(U64) * weights).sum(axis=1, dtype=U64)


def prefix_key(tokens) -> np.uint64:
    """key(p) = sum_i (token_i + 1) << 16 i  (prefix length <= 4, V <= 65535)."""
    key = 0
    for i, tok in enumerate(tokens):
        key |= (int(tok) + 1) << (16 * i)
    return U64(key)


def prefix_keys(prefixes: np.ndarray) -> np.ndarray:
    """Vectorised `prefix_key` over int rows [n, len]."""
    prefixes = np.asarray(prefixes, dtype=np.int64)
    keys = np.zeros(prefixes.shape[0], dtype=U64)
    for i in range(prefixes.shape[1]):
        keys |= (prefixes[:, i] + 1).astype(U64) << U64(16 * i)
    return keys


def mix64(key: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on uint64 (wrapping arithmetic)."""
    with np.errstate(over="ignore"):
        z = np.asarray(key, dtype=U64) + U64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> U64(30))) * U64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> U64(27))) * U64(0x94D049BB133111EB)
        z = z ^ (z >> U64(31))
    return z


def bloom_probe_positions(keys: np.ndarray, log2_bits: int, n_hashes: int) -> np.ndarray:
    """int64 [n, n_hashes]: bit positions probed for each key."""
    z = mix64(np.atleast_1d(keys))
    h1 = (z & U64(0xFFFFFFFF)).astype(np.int64)
    h2 = ((z >> U64(32)) | U64(1)).astype(np.int64)
    i = np.arange(n_hashes, dtype=np.int64)[None, :]
    pos32 = (h1[:, None] + i * h2[:, None]) & 0xFFFFFFFF
    return pos32 & ((1 << log2_bits) - 1)


class PrefixBloom:
    """One request's Bloom filter over prefix keys: m = 2**log2_bits bits, k probes."""

    def __init__(self, log2_bits: int, n_hashes: int):
        self.log2_bits = int(log2_bits)
        self.n_hashes = int(n_hashes)
        self.words = np.zeros((1 << log2_bits) // 64, dtype=U64)

    def add(self, keys: np.ndarray) -> None:
        pos = bloom_probe_positions(keys, self.log2_bits, self.n_hashes).ravel()
        np.bitwise_or.at(self.words, pos >> 6, U64(1) << (pos & 63).astype(U64))

    def contains(self, keys: np.ndarray) -> np.ndarray:
        pos = bloom_probe_positions(keys, self.log2_bits, self.n_hashes)
        bit = (self.words[pos >> 6] >> (pos & 63).astype(U64)) & U64(1)
        return np.all(bit == U64(1), axis=1)

    def fill(self) -> float:
        return float(np.unpackbits(self.words.view(np.uint8)).mean())


def build_prefix_bloom(sids: np.ndarray, eligible: np.ndarray, log2_bits: int,
                       n_hashes: int) -> PrefixBloom:
    """Insert the key of every prefix (length 1..L) of every eligible SID."""
    bloom = PrefixBloom(log2_bits, n_hashes)
    chosen = np.asarray(sids)[np.asarray(eligible, dtype=bool)]
    for l in range(1, chosen.shape[1] + 1):
        bloom.add(prefix_keys(np.unique(chosen[:, :l], axis=0)))
    return bloom


# ---------------------------------------------------------------------------
# Per-node matcher index of the paper (Sections 4.2-4.4, Appendix A)
# ---------------------------------------------------------------------------
class NodeMatcherIndex:
    """bitmask_index / bloom_index per child entry and the deduplicated row tables.

    Every trie node stores the OR of the rows of the ads below it (Section 4.2, 4.3); a child entry
    carries the ids of its child node's two rows in tables of unique rows (Section 4.4).  Built here
    from the definition: for every node, OR the rows of every ad whose SID has the node's prefix.
    """

    def __init__(self, trie, sids: np.ndarray, ad_sid: np.ndarray, ad_bitmask: np.ndarray, ad_bloom: np.ndarray):
        L = trie.sid_length
        # rows of the SIDs (leaf level): OR over the SID's ads
        order = np.argsort(ad_sid, kind="stable")
        starts = np.searchsorted(ad_sid[order], np.arange(sids.shape[0]))
        leaf_bm = np.bitwise_or.reduceat(ad_bitmask[order], starts, axis=0)
        leaf_bl = np.bitwise_or.reduceat(ad_bloom[order], starts, axis=0)
        node_bm = np.zeros((trie.num_nodes, ad_bitmask.shape[1]), dtype=U64)
        node_bl = np.zeros((trie.num_nodes, ad_bloom.shape[1]), dtype=U64)
        for l in range(L, -1, -1):
            # SIDs are sorted, so the SIDs under the i-th prefix of level l are one contiguous run
            if l == 0:
                first = np.zeros(1, dtype=np.int64)
            else:
                change = np.any(sids[1:, :l] != sids[:-1, :l], axis=1)
                first = np.concatenate([[0], np.nonzero(change)[0] + 1])
            base = int(trie.level_start[l])
            node_bm[base: base + first.shape[0]] = np.bitwise_or.reduceat(leaf_bm, first, axis=0)
            node_bl[base: base + first.shape[0]] = np.bitwise_or.reduceat(leaf_bl, first, axis=0)
        self.node_bitmask, self.node_bloom = node_bm, node_bl
        child = trie.csr_child_nodes.astype(np.int64)
        self.bitmask_table, self.bitmask_index = np.unique(node_bm[child], axis=0, return_inverse=True)
        self.bloom_table, self.bloom_index = np.unique(node_bl[child], axis=0, return_inverse=True)
        self.bitmask_index = self.bitmask_index.reshape(-1).astype(np.int32)
        self.bloom_index = self.bloom_index.reshape(-1).astype(np.int32)


class NodeRowsMatcher:
    """TM of the paper's form for `oracle.gtm.gtm_mask`: attribute bitmask AND any-location Bloom."""

    def __init__(self, trie, index: NodeMatcherIndex, user_bitmask: np.ndarray, user_blooms: np.ndarray):
        self.trie, self.index = trie, index
        self.user_bitmask, self.user_blooms = user_bitmask, user_blooms

    def match(self, request, row_key, prefix_len, tokens, child_nodes):
        out = np.zeros(tokens.shape[0], dtype=bool)
        for i, child in enumerate(child_nodes):
            j = int(child) - 1                       # child entry of node `child` (entries follow node order)
            assert int(self.trie.csr_child_nodes[j]) == int(child)
            bm = self.index.bitmask_table[self.index.bitmask_index[j]]
            bl = self.index.bloom_table[self.index.bloom_index[j]]
            out[i] = bitmask_match(bm, self.user_bitmask[request]) and bloom_any(bl, self.user_blooms[request])
        return out
