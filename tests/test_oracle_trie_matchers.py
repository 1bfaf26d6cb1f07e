"""Pins for oracle.sid_trie and oracle.matchers: brute force against python
sets, the paper's printed bitmask example, Bloom-filter invariants.  CPU only."""
import math
import os

import numpy as np
import pytest

import synth
from oracle import matchers as Mx
from oracle.sid_trie import SidTrie


@pytest.fixture(scope="module")
def small():
    rng = synth.rng_for(1, 7)
    V, L = 64, 3
    sids = synth.catalog(rng, 500, V, L)
    return sids, V, L, SidTrie(sids, V)


def test_catalog_generator_properties():
    rng = synth.rng_for(1, 1)
    sids = synth.catalog(rng, 2000, 64, 3)
    assert sids.shape == (2000, 3) and sids.dtype == np.int32
    assert len({tuple(s) for s in sids.tolist()}) == 2000
    assert sids.min() >= 0 and sids.max() < 64
    assert sids.tolist() == sorted(sids.tolist())
    full = synth.catalog(synth.rng_for(1, 2), 8, 2, 3)           # the whole space
    assert len({tuple(s) for s in full.tolist()}) == 8


def test_trie_equals_set_of_prefixes(small):
    sids, V, L, trie = small
    prefixes = {tuple(s[:l]) for s in sids.tolist() for l in range(L + 1)}
    assert trie.num_nodes == len(prefixes)
    # every inserted SID is found, and walk() agrees with set membership on random probes
    for s in sids.tolist():
        assert trie.walk(s) >= 0
    rng = np.random.default_rng(0)
    for _ in range(2000):
        l = int(rng.integers(1, L + 1))
        p = tuple(int(x) for x in rng.integers(0, V, size=l))
        assert (trie.walk(p) >= 0) == (p in prefixes)
    # every root-to-leaf path is an inserted SID; node ids are level-ordered with sorted children
    seen = set()
    stack = [(0, ())]
    while stack:
        node, pref = stack.pop()
        assert trie.prefix_of(node) == pref
        toks, kids = trie.lookup(node)
        assert toks.tolist() == sorted(toks.tolist())
        assert kids.tolist() == list(range(int(kids[0]), int(kids[0]) + len(kids))) if len(kids) else True
        if len(pref) == L:
            assert len(toks) == 0
            seen.add(pref)
        for tok, kid in zip(toks.tolist(), kids.tolist()):
            assert trie.level_of(kid) == len(pref) + 1
            stack.append((kid, pref + (tok,)))
    assert seen == {tuple(s) for s in sids.tolist()}
    assert trie.num_child_entries == trie.num_nodes - 1


def test_dense_bitmask_form_equals_csr_form(small):
    sids, V, L, trie = small
    bits, base = trie.dense_child_bits()
    bits_fast, base_fast = trie.dense_child_bits_fast()
    assert np.array_equal(bits, bits_fast) and np.array_equal(base, base_fast)
    for n in range(trie.num_internal_nodes()):
        toks, kids = trie.lookup(n)
        got = [v for v in range(V) if (int(bits[n, v // 64]) >> (v % 64)) & 1]
        assert got == toks.tolist()
        for tok, kid in zip(toks.tolist(), kids.tolist()):
            below = sum((int(bits[n, w]) & ((1 << 64) - 1 if w < tok // 64 else (1 << (tok % 64)) - 1)).bit_count()
                        for w in range(tok // 64 + 1))
            assert base[n] + below == kid


def _bits(s):
    """Bit string as printed (left to right) -> one uint64 word, leftmost char = bit 0."""
    return np.array([sum(1 << i for i, c in enumerate(s) if c == "1")], dtype=np.uint64)


def test_bitmask_worked_example(golden_dir):
    rows, expect = {}, {}
    for line in open(os.path.join(golden_dir, "bitmask_toy_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        parts = line.split()
        if parts[0] == "expect":
            expect[parts[1]] = parts[2] == "passes"
        else:
            rows[parts[0]] = _bits(parts[1] + parts[2])
    user = rows["user_us_age30"]
    assert np.array_equal(Mx.union_rows(np.stack([rows["ad_us_18_24"], rows["ad_ca_25_34"]])), rows["node_union"])
    for name, want in expect.items():
        assert Mx.bitmask_match(rows[name], user) == want, name
    # an empty user mask constrains nothing; a user bit missing from the node fails
    assert Mx.bitmask_match(rows["node_union"], _bits("00000"))
    assert not Mx.bitmask_match(rows["node_union"], _bits("00100"))
    # multi-word rows: a failure in any word fails the test
    node = np.array([0xFF, 0x0F], dtype=np.uint64)
    assert Mx.bitmask_match(node, np.array([0x81, 0x01], dtype=np.uint64))
    assert not Mx.bitmask_match(node, np.array([0x81, 0x10], dtype=np.uint64))


def test_bloom_containment_and_any():
    stored = np.array([0b1011, 0b0100, 0, 1 << 63], dtype=np.uint64)
    assert Mx.bloom_contains(stored, np.array([0b0011, 0b0100, 0, 0], dtype=np.uint64))
    assert not Mx.bloom_contains(stored, np.array([0b0111, 0, 0, 0], dtype=np.uint64))
    assert Mx.bloom_any(stored, [np.array([0b0100, 0, 0, 0], dtype=np.uint64),
                                 np.array([0b0001, 0, 0, 1 << 63], dtype=np.uint64)])
    assert not Mx.bloom_any(stored, [])
    # OR-union of rows is conservative: whatever one ad's row contains, the union contains
    rng = np.random.default_rng(3)
    ads = rng.integers(0, 2 ** 63, size=(6, 4), dtype=np.uint64) & rng.integers(0, 2 ** 63, size=(6, 4), dtype=np.uint64)
    union = Mx.union_rows(ads)
    for a in ads:
        loc = a & rng.integers(0, 2 ** 63, size=4, dtype=np.uint64)
        assert Mx.bloom_contains(a, loc) and Mx.bloom_contains(union, loc)


def test_paper_lookup_equals_filtering_children(small):
    sids, V, L, trie = small
    rng = np.random.default_rng(5)
    E = trie.num_child_entries
    bm_table = rng.integers(0, 2 ** 8, size=(17, 2), dtype=np.uint64)
    bl_table = rng.integers(0, 2 ** 16, size=(13, 4), dtype=np.uint64)
    bm_idx = rng.integers(0, 17, size=E)
    bl_idx = rng.integers(0, 13, size=E)
    user_bm = np.array([0b101, 0b1], dtype=np.uint64)
    user_bl = [rng.integers(0, 2 ** 16, size=4, dtype=np.uint64) & rng.integers(0, 2 ** 16, size=4, dtype=np.uint64)
               for _ in range(5)]
    for node in [0, 1, 5, 70]:
        got = Mx.paper_lookup(trie, bm_idx, bl_idx, bm_table, bl_table, node, user_bm, user_bl)
        want = []
        for j in range(int(trie.node_offsets[node]), int(trie.node_offsets[node + 1])):
            bm, bl = bm_table[bm_idx[j]], bl_table[bl_idx[j]]
            ok = all(int(a) & int(u) == int(u) for a, u in zip(bm, user_bm))
            ok = ok and any(all(int(q) & int(b) == int(q) for q, b in zip(row, bl)) for row in user_bl)
            if ok:
                want.append((int(trie.csr_tokens[j]), int(trie.csr_child_nodes[j])))
        assert got == want
    assert Mx.paper_lookup(trie, bm_idx, bl_idx, bm_table, bl_table, 0, user_bm, []) == []


def test_splitmix64_reference_vectors(golden_dir):
    want = [int(l, 16) for l in open(os.path.join(golden_dir, "splitmix64_vectors.txt")) if l.startswith("0x")]
    gamma = 0x9E3779B97F4A7C15
    states = np.array([(n * gamma) % 2 ** 64 for n in range(len(want))], dtype=np.uint64)
    assert [int(x) for x in Mx.mix64(states)] == want


def test_prefix_key_and_probe_positions():
    assert int(Mx.prefix_key([])) == 0
    assert int(Mx.prefix_key([0])) == 1
    assert int(Mx.prefix_key([5, 0, 1023])) == 6 + (1 << 16) + (1024 << 32)
    pref = np.array([[5, 0, 1023], [63, 63, 63]])
    assert [int(k) for k in Mx.prefix_keys(pref)] == [int(Mx.prefix_key(p)) for p in pref]
    # probes restated with python integers
    key = int(Mx.prefix_key([7, 9]))
    z = (key + 0x9E3779B97F4A7C15) % 2 ** 64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) % 2 ** 64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) % 2 ** 64
    z ^= z >> 31
    h1, h2 = z & 0xFFFFFFFF, (z >> 32) | 1
    want = [((h1 + i * h2) % 2 ** 32) % 2 ** 22 for i in range(4)]
    assert Mx.bloom_probe_positions(np.array([key], dtype=np.uint64), 22, 4)[0].tolist() == want


def test_prefix_bloom_no_false_negatives_and_fp_rate():
    rng = synth.rng_for(4, 3)
    V, L, n = 256, 4, 20000
    sids = synth.catalog(rng, n, V, L)
    elig = synth.eligible_subset(rng, n, 0.2)
    log2m, k = 18, 4
    bloom = Mx.build_prefix_bloom(sids, elig, log2m, k)
    inserted = set()
    for l in range(1, L + 1):
        keys = Mx.prefix_keys(np.unique(sids[elig][:, :l], axis=0))
        assert bloom.contains(keys).all()                      # no false negatives
        inserted.update(int(x) for x in keys)
    # false-positive rate on keys never inserted vs the analytic (1 - exp(-kn/m))^k
    probe = Mx.prefix_keys(rng.integers(0, V, size=(200000, 4)))
    fresh = np.array([int(x) not in inserted for x in probe])
    rate = bloom.contains(probe[fresh]).mean()
    m = 1 << log2m
    expect = (1 - math.exp(-k * len(inserted) / m)) ** k
    sigma = math.sqrt(expect * (1 - expect) / fresh.sum())
    assert abs(rate - expect) < 4 * sigma + 0.1 * expect
    assert abs(bloom.fill() - (1 - math.exp(-k * len(inserted) / m))) < 0.01


def test_node_eligibility_is_existence_of_eligible_descendant(small):
    sids, V, L, trie = small
    elig = synth.eligible_subset(synth.rng_for(1, 9), sids.shape[0], 0.3)
    marks = Mx.node_eligibility(trie, sids, elig)
    good = [tuple(s) for s, e in zip(sids.tolist(), elig) if e]
    for node in range(trie.num_nodes):
        p = trie.prefix_of(node)
        assert marks[node] == any(s[:len(p)] == p for s in good)
    words = Mx.pack_node_bits(marks)
    for node in range(trie.num_nodes):
        assert ((int(words[node >> 6]) >> (node & 63)) & 1) == int(marks[node])


def test_node_rows_index_is_the_union_over_descendant_ads_and_is_conservative():
    """Per-node rows = OR over the ads below the node (Sections 4.2, 4.3): brute force; and the node-level
    test never drops a prefix that has a truly eligible ad below it (it may keep more: OR-union and Bloom
    collisions are false positives only)."""
    V, L, n = 64, 3, 300
    rng = synth.rng_for(4, 70)
    sids = synth.catalog(rng, n, V, L)
    trie = SidTrie(sids, V)
    layout = synth.TargetingLayout(W_bm=2, W_bl=4, attributes=((0, 20), (20, 4), (24, 30), (64, 40)),
                                   n_locations=300, bits_per_location=3)
    loc_rows = synth.location_rows(rng, layout)
    ad_sid, ad_bm, ad_bl = synth.ads_for_sids(rng, n, layout, loc_rows)
    assert np.bincount(ad_sid, minlength=n).min() >= 1
    index = Mx.NodeMatcherIndex(trie, sids, ad_sid, ad_bm, ad_bl)
    # brute-force union per node
    for node in range(trie.num_nodes):
        p = trie.prefix_of(node)
        below = [a for a in range(ad_sid.shape[0]) if tuple(sids[ad_sid[a]][:len(p)]) == p]
        assert np.array_equal(index.node_bitmask[node], Mx.union_rows(ad_bm[below]))
        assert np.array_equal(index.node_bloom[node], Mx.union_rows(ad_bl[below]))
    # the tables are deduplicated and the indices reproduce the child's rows
    assert len({r.tobytes() for r in index.bitmask_table}) == index.bitmask_table.shape[0]
    for j in range(trie.num_child_entries):
        child = int(trie.csr_child_nodes[j])
        assert np.array_equal(index.bitmask_table[index.bitmask_index[j]], index.node_bitmask[child])
        assert np.array_equal(index.bloom_table[index.bloom_index[j]], index.node_bloom[child])
    # conservativeness against exact ad-level matching
    ubm, ubl, uloc = synth.request_attributes(rng, 4, layout, loc_rows, n_loc=8)
    for b in range(4):
        eligible_ads = [a for a in range(ad_sid.shape[0])
                        if Mx.bitmask_match(ad_bm[a], ubm[b]) and Mx.bloom_any(ad_bl[a], ubl[b])]
        for a in eligible_ads:
            sid = sids[ad_sid[a]]
            for l in range(1, L + 1):
                node = trie.walk(sid[:l])
                assert Mx.bitmask_match(index.node_bitmask[node], ubm[b])
                assert Mx.bloom_any(index.node_bloom[node], ubl[b])
        # Appendix A lookup from the root = the children whose rows pass
        got = Mx.paper_lookup(trie, index.bitmask_index, index.bloom_index, index.bitmask_table, index.bloom_table,
                              0, ubm[b], ubl[b])
        want = [(int(t), int(c)) for t, c in zip(*trie.lookup(0))
                if Mx.bitmask_match(index.node_bitmask[c], ubm[b]) and Mx.bloom_any(index.node_bloom[c], ubl[b])]
        assert got == want


def test_gtm_mask_with_node_rows_matcher_equals_the_appendix_a_lookup():
    """`NodeRowsMatcher` plugged into `gtm_mask` must allow, for every beam, exactly the (token, child)
    pairs the Appendix A lookup emits for that beam's node and that beam's request; and the candidate
    score of such a pair is the beam's score plus the token's log-probability (Section 4.1)."""
    V, L, n = 64, 3, 300
    rng = synth.rng_for(4, 71)
    sids = synth.catalog(rng, n, V, L)
    trie = SidTrie(sids, V)
    layout = synth.TargetingLayout(W_bm=2, W_bl=4, attributes=((0, 20), (20, 4), (24, 30), (64, 40)),
                                   n_locations=300, bits_per_location=3)
    loc_rows = synth.location_rows(rng, layout)
    ad_sid, ad_bm, ad_bl = synth.ads_for_sids(rng, n, layout, loc_rows)
    index = Mx.NodeMatcherIndex(trie, sids, ad_sid, ad_bm, ad_bl)
    B, M = 3, 5
    ubm, ubl, _ = synth.request_attributes(rng, B, layout, loc_rows, n_loc=8)
    matcher = Mx.NodeRowsMatcher(trie, index, ubm, ubl)
    from oracle.gtm import gtm_mask
    internal = [node for node in range(trie.num_nodes) if trie.lookup(node)[0].size > 0]
    some_kept = some_dropped = False
    for depth_nodes in (internal[:1] * (B * M), internal[1:1 + B * M], internal[-B * M:]):
        beam_node = np.array(depth_nodes, dtype=np.int64)
        beam_node[2] = -1                                         # a dead beam allows nothing
        score = -np.arange(B * M, dtype=np.float32)
        logp = np.log(np.full((B * M, V), 1.0 / V, dtype=np.float32)) - 0.01 * np.arange(V, dtype=np.float32)
        cand, allow, child = gtm_mask(logp, score, beam_node, np.zeros(B * M, dtype=np.uint64), 0, trie, matcher, B, M)
        for r in range(B * M):
            if beam_node[r] < 0:
                assert not allow[r].any() and np.isneginf(cand[r]).all()
                continue
            b = r // M
            want = Mx.paper_lookup(trie, index.bitmask_index, index.bloom_index, index.bitmask_table,
                                   index.bloom_table, int(beam_node[r]), ubm[b], ubl[b])
            got = [(int(v), int(child[r, v])) for v in np.flatnonzero(allow[r])]
            assert got == want
            for v, _ in want:
                assert cand[r, v] == np.float32(score[r]) + logp[r, v]
            assert np.isneginf(cand[r][~allow[r]]).all()
            n_children = trie.lookup(int(beam_node[r]))[0].size
            some_kept |= len(want) > 0
            some_dropped |= len(want) < n_children
    assert some_kept and some_dropped                             # the comparison saw both outcomes
