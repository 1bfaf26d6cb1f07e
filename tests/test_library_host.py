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


def test_layer_norm_fold_and_centring_helpers(api):
    """The host-side weight preparation of the folded-LayerNorm path against its definition in fp64:
    with the helper's outputs, rstd * (x @ w'^T) - rstd * mean * col_sum + col_bias equals LayerNorm(x) @ w^T up
    to the one bf16 rounding of w * gamma; centred rows / outputs have zero mean along the stream's feature
    axis and differ from the input by exactly that mean; and running the oracle's decoder on weights centred
    by the helpers changes no log-probability (the identity the product path relies on)."""
    rng = synth.rng_for(1, 901)
    N, K, R = 96, 160, 40
    w = synth.normal_f32(rng, (N, K)) * 0.3
    gamma = (1.0 + 0.3 * synth.normal_f32(rng, K)).astype(np.float32)
    beta = (0.4 * synth.normal_f32(rng, K)).astype(np.float32)
    x = (synth.normal_f32(rng, (R, K)) * 2.0 + 0.7).astype(np.float64)
    wf_bits, cs, cb = api.grace_fold_layer_norm(w, gamma, beta)
    wf = synth.bf16_bits_to_f32(wf_bits).astype(np.float64)
    exact = w.astype(np.float64) * gamma.astype(np.float64)[None, :]
    assert (np.abs(wf - exact) <= 2.0 ** -8 * np.abs(exact)).all()               # one rounding to bf16 (half an ulp of 8 bits)
    assert np.array_equal(wf_bits, synth.f32_to_bf16_bits((w * gamma[None, :]).astype(np.float32)))
    np.testing.assert_allclose(cs, wf.sum(axis=1), rtol=1e-6, atol=1e-6)         # sums of the ROUNDED operands
    np.testing.assert_allclose(cb, w.astype(np.float64) @ beta.astype(np.float64), rtol=1e-6, atol=1e-6)
    mean, var = x.mean(axis=1, keepdims=True), x.var(axis=1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + 1e-5)
    ln = (x - mean) * rstd * gamma[None, :] + beta[None, :]
    folded = rstd * (x @ wf.T) - rstd * mean * cs[None, :].astype(np.float64) + cb[None, :].astype(np.float64)
    ref_rounded = ((x - mean) * rstd) @ wf.T + beta.astype(np.float64) @ w.astype(np.float64).T
    np.testing.assert_allclose(folded, ref_rounded, rtol=0, atol=2e-5)           # the identity itself (same operands)
    # and the cost of rounding w * gamma to bf16: at most 2^-8 of every product, element by element
    assert (np.abs(folded - ln @ w.astype(np.float64).T) <= 2.0 ** -8 * (np.abs((x - mean) * rstd) @ np.abs(exact).T) + 1e-6).all()
    # centring
    a = (synth.normal_f32(rng, (50, K)) + 1.5).astype(np.float32)
    ca = api.grace_centre_rows(a)
    np.testing.assert_allclose(ca.astype(np.float64).mean(axis=1), 0.0, atol=1e-6)
    np.testing.assert_allclose(ca, a.astype(np.float64) - a.astype(np.float64).mean(axis=1, keepdims=True), rtol=0, atol=1e-6)
    wo = (synth.normal_f32(rng, (K, 70)) + 0.3).astype(np.float32)               # [stream features, inputs]
    co = api.grace_centre_outputs(wo)
    np.testing.assert_allclose(co.astype(np.float64).mean(axis=0), 0.0, atol=1e-6)
    np.testing.assert_allclose(co, wo.astype(np.float64) - wo.astype(np.float64).mean(axis=0, keepdims=True), rtol=0, atol=1e-6)
    h = synth.normal_f32(rng, (9, 70)).astype(np.float64)
    np.testing.assert_allclose((h @ co.astype(np.float64).T).mean(axis=1), 0.0, atol=1e-5)   # outputs have zero mean
    bits = api.grace_f32_to_bf16(a)
    assert np.array_equal(bits, synth.f32_to_bf16_bits(a))
    # the oracle's decoder on helper-centred weights: no log-probability moves
    import copy
    from oracle import decoder as D
    shp = synth.DecoderShape(2, 64, 4, 16, 128, 48, 32, 3)
    wts = synth.decoder_weights(synth.rng_for(1, 902), shp, std=0.2, as_bf16=False)
    wts["embed"] = np.asarray(wts["embed"], np.float64) + 1.5
    enc = synth.normal_f32(rng, (2, 10, 48)).astype(np.float64)

    def log_probs(wd):
        state = D.DecoderState(shp, 2, [1, 1])
        return D.decoder_forward(wd, shp, state, D.cross_kv(wd, shp, enc), np.full(2, shp.V), 0, 2)
    c = copy.deepcopy(wts)
    c["embed"] = api.grace_centre_rows(c["embed"]).astype(np.float64)
    c["pos"] = api.grace_centre_rows(c["pos"]).astype(np.float64)
    for lw in c["layers"]:
        for name in ("w_o", "w_oc", "w_2"):
            lw[name] = api.grace_centre_outputs(lw[name]).astype(np.float64)
    np.testing.assert_allclose(log_probs(c), log_probs(wts), rtol=0, atol=2e-5)  # fp32 storage of the centred weights
