"""CPU-only checks of the C-ABI library: it builds, loads, exports every symbol
the header declares, validates arguments, and its host-side index builders
agree bit for bit with the oracle's independently built structures."""
import ctypes
import os
import re

import numpy as np
import pytest

import synth
from oracle import matchers as Mx
from oracle.sid_trie import SidTrie

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def api():
    from paper_2608_00938_b200 import build
    build()
    from paper_2608_00938_b200 import api as _api
    return _api


def test_every_declared_symbol_is_exported(api):
    header = open(os.path.join(ROOT, "include", "grace.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(grace_[a-z0-9_]+)\s*\(", header))
    assert {"grace_cross_attn", "grace_self_attn", "grace_gtm_mask", "grace_beam_topk",
            "grace_decode_step"} <= declared
    for name in sorted(declared):
        assert hasattr(api.lib, name), f"{name} declared in grace.h but not exported"
    assert api.version() >= 1 and api.built_for_sm() == 100


def test_struct_layouts_match_the_header(api):
    # sizes computed from the C declarations: a drift between grace.h and the binding shows here
    assert ctypes.sizeof(api.TrieStruct) == 4 + 4 + 8 + 8 + 8 + 8
    assert ctypes.sizeof(api.MatcherStruct) == 4 * 4 + 8 + 8
    assert ctypes.sizeof(api.LayerStruct) == 23 * 8


def test_host_argument_validation(api):
    sids = np.array([[1, 2], [1, 2]], dtype=np.int32)            # duplicate
    with pytest.raises(api.GraceError):
        api.grace_trie_count_nodes(sids, 64)
    unsorted = np.array([[3, 2], [1, 2]], dtype=np.int32)
    with pytest.raises(api.GraceError):
        api.grace_trie_count_nodes(unsorted, 64)
    with pytest.raises(api.GraceError):
        api.grace_trie_count_nodes(np.array([[1, 70]], dtype=np.int32), 64)     # token out of range
    assert api.grace_beam_topk_workspace_bytes(32, 1 << 21, 2048) > 0
    # null device pointers are rejected on the host before anything is launched
    assert api.lib.grace_self_attn(None, 0, None, None, None, None, None, 0, 1, 0, 8, 64, 16, 0.125, None, None) == 1
    assert api.lib.grace_beam_topk(None, 1, 16, 4, 4, None, None, None, None, None, 0, None, None) == 1
    assert api.lib.grace_decode_step(None, 0, None) == 1


@pytest.mark.parametrize("V,L,n", [(64, 3, 2000), (128, 4, 5000), (64, 1, 40), (64, 2, 300)])
def test_dense_trie_builder_matches_oracle(api, V, L, n):
    sids = synth.catalog(synth.rng_for(1, 50 + L), n, V, L)
    trie = SidTrie(sids, V)
    bits, base, level_start = api.grace_trie_build_dense(sids, V)
    assert level_start.tolist() == trie.level_start.tolist()
    o_bits, o_base = trie.dense_child_bits_fast()
    assert np.array_equal(bits, o_bits)
    assert np.array_equal(base, o_base)
    rng = np.random.default_rng(0)
    for _ in range(300):
        l = int(rng.integers(0, L + 1))
        if rng.random() < 0.5:
            p = sids[rng.integers(0, n), :l]
        else:
            p = rng.integers(0, V, size=l)
        assert api.grace_trie_walk(bits, base, V, L, p) == trie.walk(p)


def test_matcher_builders_match_oracle(api):
    V, L, n = 128, 4, 6000
    rng = synth.rng_for(4, 60)
    sids = synth.catalog(rng, n, V, L)
    elig = synth.eligible_subset(rng, n, 0.2)
    trie = SidTrie(sids, V)
    got = api.grace_node_bitmask_build(sids, V, elig, trie.num_nodes)
    want = Mx.pack_node_bits(Mx.node_eligibility(trie, sids, elig))
    assert np.array_equal(got, want)
    for log2m, k in [(16, 4), (12, 3), (20, 7)]:
        words = api.grace_bloom_build(sids, V, elig, log2m, k)
        assert np.array_equal(words, Mx.build_prefix_bloom(sids, elig, log2m, k).words)
    none = api.grace_node_bitmask_build(sids, V, np.zeros(n, bool), trie.num_nodes)
    assert not none.any()


def test_gtm_index_builder_matches_oracle_rows(api):
    """The library's host builder of the per-node matcher index (Appendix A layout) against the oracle's:
    same CSR arrays; same row content behind every child entry's two indices; tables free of duplicates."""
    V, L, n = 128, 4, 4000
    rng = synth.rng_for(4, 80)
    sids = synth.catalog(rng, n, V, L)
    trie = SidTrie(sids, V)
    layout = synth.TargetingLayout()
    loc_rows = synth.location_rows(rng, layout)
    ad_sid, ad_bm, ad_bl = synth.ads_for_sids(rng, n, layout, loc_rows)
    ref = Mx.NodeMatcherIndex(trie, sids, ad_sid, ad_bm, ad_bl)
    got = api.grace_gtm_index_build(sids, V, ad_sid, ad_bm, ad_bl)
    assert got["num_nodes"] == trie.num_nodes
    assert np.array_equal(got["node_offsets"], trie.node_offsets)
    assert np.array_equal(got["csr_child_nodes"], trie.csr_child_nodes)
    assert np.array_equal(got["csr_tokens"], trie.csr_tokens)
    assert np.array_equal(got["bitmask_table"][got["bitmask_index"]], ref.bitmask_table[ref.bitmask_index])
    assert np.array_equal(got["bloom_table"][got["bloom_index"]], ref.bloom_table[ref.bloom_index])
    assert got["bitmask_table"].shape == ref.bitmask_table.shape and got["bloom_table"].shape == ref.bloom_table.shape
    assert len({r.tobytes() for r in got["bloom_table"]}) == got["bloom_table"].shape[0]
    # unsorted ads are rejected
    with pytest.raises(api.GraceError):
        api.grace_gtm_index_build(sids, V, ad_sid[::-1].copy(), ad_bm, ad_bl)


@pytest.mark.parametrize("policy", [("static", [0, 4, 2, 2, 1]), ("dynamic", 0.35, 6)])
def test_kway_index_builder_matches_oracle(api, policy):
    """k-way partitioned rows (Section 4.2): the library's host builder against the oracle's, slot by slot."""
    from oracle import kway as KW
    V, L, n = 64, 4, 1500
    rng = synth.rng_for(4, 81)
    sids = synth.catalog(rng, n, V, L)
    trie = SidTrie(sids, V)
    layout = synth.TargetingLayout()
    loc_rows = synth.location_rows(rng, layout)
    ad_sid, ad_bm, ad_bl = synth.ads_for_sids(rng, n, layout, loc_rows)
    ref = KW.KWayMatcherIndex(trie, sids, ad_sid, ad_bm, ad_bl, policy)
    if policy[0] == "static":
        got = api.grace_gtm_index_build_kway(sids, V, ad_sid, ad_bm, ad_bl, k_level=policy[1])
    else:
        got = api.grace_gtm_index_build_kway(sids, V, ad_sid, ad_bm, ad_bl, fill_target=policy[1], k_max=policy[2])
    assert np.array_equal(got["node_offsets"], trie.node_offsets)
    assert np.array_equal(got["csr_tokens"], trie.csr_tokens)
    assert np.array_equal(got["part_offsets"], ref.part_offsets)
    assert (np.diff(got["part_offsets"]) > 1).any()                  # some node really is partitioned
    assert np.array_equal(got["bitmask_table"][got["bitmask_index"]], ref.part_bitmask_rows)
    assert np.array_equal(got["bloom_table"][got["bloom_index"]], ref.part_bloom_rows)
    assert got["bitmask_table"].shape == ref.bitmask_table.shape and got["bloom_table"].shape == ref.bloom_table.shape
    # k = 1 everywhere is the unpartitioned index
    one = api.grace_gtm_index_build_kway(sids, V, ad_sid, ad_bm, ad_bl, k_level=[1] * (L + 1))
    plain = api.grace_gtm_index_build(sids, V, ad_sid, ad_bm, ad_bl)
    assert np.array_equal(one["part_offsets"], np.arange(trie.num_nodes))
    assert np.array_equal(one["bitmask_table"][one["bitmask_index"]], plain["bitmask_table"][plain["bitmask_index"]])
    with pytest.raises(api.GraceError):
        api.grace_gtm_index_build_kway(sids, V, ad_sid, ad_bm, ad_bl, k_level=[0] * (L + 1))
