"""Pins of the k-way partitioned matcher oracle (Section 4.2 "k-way partition", Sections 4.3, 4.4)."""
import os

import numpy as np
import pytest

import synth
from oracle import kway as KW
from oracle import matchers as Mx
from oracle.sid_trie import SidTrie


def _setup(n=300, V=64, L=3, variant=80, n_req=4):
    rng = synth.rng_for(4, variant)
    sids = synth.catalog(rng, n, V, L)
    trie = SidTrie(sids, V)
    layout = synth.TargetingLayout(W_bm=2, W_bl=4, attributes=((0, 20), (20, 4), (24, 30), (64, 40)),
                                   n_locations=300, bits_per_location=3)
    loc_rows = synth.location_rows(rng, layout)
    ad_sid, ad_bm, ad_bl = synth.ads_for_sids(rng, n, layout, loc_rows)
    ubm, ubl, _ = synth.request_attributes(rng, n_req, layout, loc_rows, n_loc=8)
    return dict(sids=sids, trie=trie, ad_sid=ad_sid, ad_bm=ad_bm, ad_bl=ad_bl, ubm=ubm, ubl=ubl, L=L)


def _bits(s):
    v = 0
    for i, c in enumerate(s):
        if c == "1":
            v |= 1 << i
    return np.array([v], dtype=np.uint64)


def test_worked_example_is_filtered_once_its_two_ads_sit_in_different_groups(golden_dir):
    """Section 4.2 prints a node whose union row passes for a user although neither ad does; that is the
    false positive k-way partitioning is there to remove: with two groups the user must fail."""
    rows = {}
    for line in open(os.path.join(golden_dir, "bitmask_toy_example.txt")):
        if line.startswith("#") or not line.strip() or line.startswith("expect"):
            continue
        name, country, age = line.split()
        rows[name] = _bits(country + age)
    bm = np.stack([rows["ad_us_18_24"], rows["ad_ca_25_34"]])
    bl = np.zeros((2, 1), dtype=np.uint64)                      # no location attribute in the example
    user, no_loc = rows["user_us_age30"], np.zeros((1, 1), dtype=np.uint64)
    g_bm, g_bl = KW.greedy_groups(bm, bl, 1)
    assert g_bm.shape[0] == 1 and np.array_equal(g_bm[0], rows["node_union"])
    assert Mx.bitmask_match(g_bm[0], user)                      # one group: kept (the paper's outcome)
    g_bm, g_bl = KW.greedy_groups(bm, bl, 2)
    assert g_bm.shape[0] == 2                                   # the second ad opens its own group (smaller fill)
    assert not any(Mx.bitmask_match(r, user) and Mx.bloom_any(q, no_loc) for r, q in zip(g_bm, g_bl))
    # a user one of the ads really serves is kept under any k
    for k in (1, 2):
        g_bm, _ = KW.greedy_groups(bm, bl, k)
        assert any(Mx.bitmask_match(r, _bits("10010")) for r in g_bm)


def test_greedy_rule_by_hand():
    # widths: 1 + 1 words.  SIDs in order; fills after the OR decide, ties go to the lowest group.
    bm = np.array([[0b0011], [0b0011], [0b1100], [0b0111]], dtype=np.uint64)
    bl = np.zeros((4, 1), dtype=np.uint64)
    g_bm, _ = KW.greedy_groups(bm, bl, 2)
    # s0 -> g0 (all empty, tie); s1 identical: g0 stays at 2 bits, g1 would get 2: tie -> g0;
    # s2: g0 would grow to 4, g1 to 2 -> g1; s3 (0111): g0 -> 3 bits, g1 -> 4 bits -> g0.
    assert [int(r[0]) for r in g_bm] == [0b0111, 0b1100]
    g_bm, _ = KW.greedy_groups(bm, bl, 8)
    assert g_bm.shape[0] <= 4 and np.array_equal(np.bitwise_or.reduce(g_bm, axis=0), np.array([0b1111], dtype=np.uint64))
    assert KW.node_fill(np.array([[0xFF]], dtype=np.uint64), np.array([[0x0F]], dtype=np.uint64)) == 12 / 128


def test_k1_is_the_unpartitioned_index():
    s = _setup()
    plain = Mx.NodeMatcherIndex(s["trie"], s["sids"], s["ad_sid"], s["ad_bm"], s["ad_bl"])
    kw = KW.KWayMatcherIndex(s["trie"], s["sids"], s["ad_sid"], s["ad_bm"], s["ad_bl"], ("static", [1] * (s["L"] + 1)))
    E = s["trie"].num_nodes - 1
    assert np.array_equal(kw.part_offsets, np.arange(E + 1))
    assert np.array_equal(kw.bitmask_table[kw.bitmask_index], plain.bitmask_table[plain.bitmask_index])
    assert np.array_equal(kw.bloom_table[kw.bloom_index], plain.bloom_table[plain.bloom_index])


@pytest.mark.parametrize("policy", [("static", [0, 4, 2, 1]), ("static", [0, 3, 3, 3]), ("dynamic", 0.30, 4),
                                    ("dynamic", 0.0, 64)])
def test_partitions_cover_the_node_never_lose_an_eligible_ad_and_only_tighten(policy):
    s = _setup()
    trie, sids = s["trie"], s["sids"]
    plain = Mx.NodeMatcherIndex(trie, sids, s["ad_sid"], s["ad_bm"], s["ad_bl"])
    kw = KW.KWayMatcherIndex(trie, sids, s["ad_sid"], s["ad_bm"], s["ad_bl"], policy)
    E = trie.num_nodes - 1
    assert kw.part_offsets[0] == 0 and (np.diff(kw.part_offsets) >= 1).all()
    leaf_bm, leaf_bl = KW.sid_rows(sids.shape[0], s["ad_sid"], s["ad_bm"], s["ad_bl"])
    for j in range(E):
        child = j + 1
        lo, hi = int(kw.part_offsets[j]), int(kw.part_offsets[j + 1])
        # the groups' rows OR back to the node's union row
        assert np.array_equal(np.bitwise_or.reduce(kw.bitmask_table[kw.bitmask_index[lo:hi]], axis=0), plain.node_bitmask[child])
        assert np.array_equal(np.bitwise_or.reduce(kw.bloom_table[kw.bloom_index[lo:hi]], axis=0), plain.node_bloom[child])
        n_below = sum(1 for i in range(sids.shape[0]) if tuple(sids[i][:len(trie.prefix_of(child))]) == trie.prefix_of(child))
        assert hi - lo <= n_below
        if policy[0] == "static":
            assert hi - lo <= policy[1][len(trie.prefix_of(child))]
        else:
            assert hi - lo <= kw.part_k[j] <= min(policy[2], n_below)
            if kw.part_k[j] < min(policy[2], n_below):      # stopped early: the target was met, and not before
                assert KW.node_fill(kw.part_bitmask_rows[lo:hi], kw.part_bloom_rows[lo:hi]) <= policy[1]
                if kw.part_k[j] > 1:
                    below = [i for i in range(sids.shape[0]) if tuple(sids[i][:len(trie.prefix_of(child))]) == trie.prefix_of(child)]
                    assert KW.node_fill(*KW.greedy_groups(leaf_bm[below], leaf_bl[below], int(kw.part_k[j]) - 1)) > policy[1]
    for b in range(s["ubm"].shape[0]):
        ubm, ubl = s["ubm"][b], s["ubl"][b]
        for j in range(E):
            child = j + 1
            kept = kw.entry_passes(j, ubm, ubl)
            union_kept = Mx.bitmask_match(plain.node_bitmask[child], ubm) and Mx.bloom_any(plain.node_bloom[child], ubl)
            assert (not kept) or union_kept                    # a group's rows are subsets of the union's
        # exact ad-level eligibility is never lost, at any prefix of the ad's SID
        for a in range(s["ad_sid"].shape[0]):
            if Mx.bitmask_match(s["ad_bm"][a], ubm) and Mx.bloom_any(s["ad_bl"][a], ubl):
                sid = sids[s["ad_sid"][a]]
                for l in range(1, s["L"] + 1):
                    assert kw.entry_passes(trie.walk(sid[:l]) - 1, ubm, ubl)
    if policy == ("dynamic", 0.0, 64):
        # one group per SID (no fill target can be met, k_max is large): the SID-level test is exact:
        # a prefix is kept iff some SID below passes on its own rows
        for b in range(s["ubm"].shape[0]):
            ubm, ubl = s["ubm"][b], s["ubl"][b]
            sid_ok = [Mx.bitmask_match(leaf_bm[i], ubm) and Mx.bloom_any(leaf_bl[i], ubl) for i in range(sids.shape[0])]
            for j in range(E):
                p = trie.prefix_of(j + 1)
                below = [i for i in range(sids.shape[0]) if tuple(sids[i][:len(p)]) == p]
                if len(below) <= 64 and len({(leaf_bm[i].tobytes(), leaf_bl[i].tobytes()) for i in below}) == len(below):
                    assert kw.entry_passes(j, ubm, ubl) == any(sid_ok[i] for i in below)


def test_more_groups_keep_fewer_prefixes_on_average():
    s = _setup(n=400, variant=81, n_req=8)
    kept = []
    for k in (1, 2, 8):
        kw = KW.KWayMatcherIndex(s["trie"], s["sids"], s["ad_sid"], s["ad_bm"], s["ad_bl"], ("static", [0, k, k, k]))
        kept.append(sum(kw.entry_passes(j, s["ubm"][b], s["ubl"][b])
                        for b in range(8) for j in range(s["trie"].num_nodes - 1)))
    assert kept[0] >= kept[1] >= kept[2] and kept[0] > kept[2]


def test_gtm_mask_with_kway_matcher_keeps_a_child_iff_one_of_its_groups_passes():
    """`KWayRowsMatcher` plugged into `gtm_mask`: a child is allowed iff at least one group of its node
    passes the bitmask test and the any-location Bloom test on its own row pair (Section 4.2, k-way
    partition), written out here directly on the index arrays."""
    from oracle.gtm import gtm_mask
    s = _setup()
    trie, sids = s["trie"], s["sids"]
    kw = KW.KWayMatcherIndex(trie, sids, s["ad_sid"], s["ad_bm"], s["ad_bl"], ("static", [0, 4, 2, 1]))
    B = s["ubm"].shape[0]
    M = 4
    matcher = KW.KWayRowsMatcher(trie, kw, s["ubm"], s["ubl"])
    internal = [node for node in range(trie.num_nodes) if trie.lookup(node)[0].size > 0]
    beam_node = np.array((internal * (B * M))[:B * M], dtype=np.int64)
    V = trie.vocab_size
    logp = -0.01 * np.arange(B * M * V, dtype=np.float32).reshape(B * M, V)
    score = -np.arange(B * M, dtype=np.float32)
    cand, allow, child = gtm_mask(logp, score, beam_node, np.zeros(B * M, dtype=np.uint64), 0, trie, matcher, B, M)
    kept = dropped = 0
    for r in range(B * M):
        b = r // M
        tokens, kids = trie.lookup(int(beam_node[r]))
        for v, c in zip(tokens, kids):
            groups = range(int(kw.part_offsets[int(c) - 1]), int(kw.part_offsets[int(c)]))
            want = any(np.array_equal(kw.bitmask_table[kw.bitmask_index[g]] & s["ubm"][b], s["ubm"][b]) and
                       any(np.array_equal(kw.bloom_table[kw.bloom_index[g]] & row, row) for row in s["ubl"][b])
                       for g in groups)
            assert bool(allow[r, v]) == want
            if want:
                assert int(child[r, v]) == int(c) and cand[r, v] == np.float32(score[r]) + logp[r, v]
            kept += want
            dropped += not want
        others = np.ones(V, dtype=bool)
        others[tokens] = False
        assert not allow[r][others].any()
    assert kept > 0 and dropped > 0
