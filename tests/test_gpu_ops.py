"""GPU parity: every C-ABI op against the oracle on the same seeded inputs, at
sizes the oracle finishes in seconds that still span several tiles and ragged
tails.  Integer / index / mask results bit-exact; bf16 attention within
2e-2 max-abs and 1e-2 relative of the fp64 oracle."""
import numpy as np
import pytest
import torch

import synth
from oracle import attention as OA
from oracle import gtm as OG
from oracle import matchers as OM
from oracle import topk as OT
from oracle.sid_trie import SidTrie

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2608_00938_b200 import api as _api
    return _api


from gpu_util import DEV, assert_attention_close, assert_gemm_close, dev, dev_bf16, f64, host_u64  # noqa: E402


# ------------------------------------------------------------------------------------------
# CD + GTM mask
# ------------------------------------------------------------------------------------------
def _mask_problem(seed, V, L, n_sids, B, M, depth, frac=0.3):
    rng = synth.rng_for(4, seed)
    sids = synth.catalog(rng, n_sids, V, L)
    trie = SidTrie(sids, V)
    elig = [synth.eligible_subset(rng, n_sids, frac) for _ in range(B)]
    prefix = np.zeros((B, M, depth), dtype=np.int32)
    node = np.full((B, M), -1, dtype=np.int32)
    for b in range(B):
        pr = synth.beam_prefixes_from_sids(rng, sids[elig[b]], depth, M) if depth else np.zeros((1, 0), np.int32)
        n = pr.shape[0]
        prefix[b, :n] = pr
        node[b, :n] = [trie.walk(p) for p in pr]
    key = OM.prefix_keys(prefix.reshape(B * M, depth))
    score = np.concatenate([synth.descending_scores(rng, M, depth) for _ in range(B)])
    logp = synth.logp_rows(rng, B * M, V)
    return sids, trie, elig, node.reshape(-1), key, score, logp


@pytest.mark.parametrize("kind", ["none", "node", "bloom"])
@pytest.mark.parametrize("V,L,n_sids,B,M,depth", [
    (64, 3, 2000, 1, 16, 1),          # config-1 sized
    (1024, 4, 60000, 3, 37, 1),       # dense level-1 rows, ragged row count
    (1024, 4, 60000, 2, 64, 2),       # sparse rows
    (2048, 4, 30000, 2, 9, 1),        # one bitmask word per lane
    (4096, 3, 30000, 2, 5, 1),        # more than one 2048-token chunk
    (192, 3, 5000, 2, 11, 0),         # root row, V not a multiple of 128
    # more than 2048 rows: warp-per-row kernel (fewer rows run a CTA per row)
    (192, 3, 5000, 3, 700, 1), (4096, 3, 30000, 2, 1030, 1), (64, 3, 2000, 5, 500, 2),
])
def test_gtm_mask_matches_oracle(api, kind, V, L, n_sids, B, M, depth):
    if depth == 0:
        M = 1
    sids, trie, elig, node, key, score, logp = _mask_problem(7 * V + depth, V, L, n_sids, B, M, depth)
    node[-1] = -1                                                     # a dead beam
    bits, base, level_start = api.grace_trie_build_dense(sids, V)
    d_bits, d_base = dev(bits), dev(base)
    trie_s = api.make_trie(d_bits, d_base, V, L, trie.num_nodes)
    if kind == "none":
        o_matcher, matcher, keep = OG.NoMatcher(), api.make_matcher(api.MATCH_NONE), None
    elif kind == "node":
        o_matcher = OG.NodeBitmaskMatcher(np.stack([OM.node_eligibility(trie, sids, e) for e in elig]))
        keep = dev(np.stack([api.grace_node_bitmask_build(sids, V, e, trie.num_nodes) for e in elig]))
        matcher = api.make_matcher(api.MATCH_NODE_BITMASK, keep)
    else:
        o_matcher = OG.PrefixBloomMatcher([OM.build_prefix_bloom(sids, e, 16, 4) for e in elig])
        keep = dev(np.stack([api.grace_bloom_build(sids, V, e, 16, 4) for e in elig]))
        matcher = api.make_matcher(api.MATCH_PREFIX_BLOOM, keep, 16, 4)
    cand_ref, allow_ref, child_ref = OG.gtm_mask(logp, score, node, key, depth, trie, o_matcher, B, M)
    cand = torch.full((B * M, V), 7.0, device=DEV)
    allow = torch.zeros((B * M, V // 64), dtype=torch.int64, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    api.grace_gtm_mask(dev(logp), dev(score), dev(node), dev(key), trie_s, matcher, cand, allow, B, M, depth, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert np.array_equal(host_u64(allow), OG.pack_allow_bits(allow_ref))
    assert np.array_equal(cand.cpu().numpy().view(np.uint32), cand_ref.view(np.uint32))      # bit-exact fp32
    # in-place form (cand aliases logp) and the mask-only form give the same result
    inplace = dev(logp)
    api.grace_gtm_mask(inplace, dev(score), dev(node), dev(key), trie_s, matcher, inplace, None, B, M, depth, status)
    assert np.array_equal(inplace.cpu().numpy().view(np.uint32), cand_ref.view(np.uint32))


@pytest.mark.parametrize("kind", ["node", "bloom"])
@pytest.mark.parametrize("V,M,depth", [(1024, 37, 1), (2048, 20, 1), (64, 16, 1), (1024, 50, 2), (192, 1100, 1),
                                       (1024, 1050, 2)])
def test_gtm_mask_logits_fused_log_softmax(api, kind, V, M, depth):
    """Fused variant: raw logits in; same allow bits as the oracle (exact), candidates equal to
    score + (logit - lse) in fp32, and the row log-sum-exp within fp32 rounding of the fp64 value."""
    L, B, n_sids = (3, 2, 2000) if V == 64 else (4, 2, 60000)
    sids, trie, elig, node, key, score, _ = _mask_problem(5 * V + depth, V, L, n_sids, B, M, depth)
    node[-1] = -1
    rng = synth.rng_for(4, 77)
    logits = synth.normal_f32(rng, (B * M, V), 3.0)
    z = logits.astype(np.float64)
    lse_ref = z.max(1) + np.log(np.exp(z - z.max(1, keepdims=True)).sum(1))
    logp_ref = (z - lse_ref[:, None]).astype(np.float32)
    bits, base, _ = api.grace_trie_build_dense(sids, V)
    trie_s = api.make_trie(dev(bits), dev(base), V, L, trie.num_nodes)
    if kind == "node":
        o_matcher = OG.NodeBitmaskMatcher(np.stack([OM.node_eligibility(trie, sids, e) for e in elig]))
        matcher = api.make_matcher(api.MATCH_NODE_BITMASK,
                                   dev(np.stack([api.grace_node_bitmask_build(sids, V, e, trie.num_nodes) for e in elig])))
    else:
        o_matcher = OG.PrefixBloomMatcher([OM.build_prefix_bloom(sids, e, 16, 4) for e in elig])
        matcher = api.make_matcher(api.MATCH_PREFIX_BLOOM, dev(np.stack([api.grace_bloom_build(sids, V, e, 16, 4) for e in elig])), 16, 4)
    cand_ref, allow_ref, _ = OG.gtm_mask(logp_ref, score, node, key, depth, trie, o_matcher, B, M)
    d_logits = dev(logits)
    cand = torch.full((B * M, V), 7.0, device=DEV)
    allow = torch.zeros((B * M, V // 64), dtype=torch.int64, device=DEV)
    lse = torch.full((B * M,), -1.0, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    api.grace_gtm_mask_logits(d_logits, lse, dev(score), dev(node), dev(key), trie_s, matcher, cand, allow, B, M, depth, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert np.array_equal(host_u64(allow), OG.pack_allow_bits(allow_ref))
    h_cand, h_lse = cand.cpu().numpy(), lse.cpu().numpy()
    live = node >= 0
    np.testing.assert_allclose(h_lse[live], lse_ref[live], atol=2e-5, rtol=0)
    assert (h_lse[~live] == 0).all()
    assert np.array_equal(np.isfinite(h_cand), allow_ref)
    np.testing.assert_allclose(h_cand[allow_ref], cand_ref[allow_ref], atol=3e-5, rtol=0)
    own = (score[:, None] + (logits - h_lse[:, None]))[allow_ref]                 # the kernel's own fp32 arithmetic
    assert np.array_equal(h_cand[allow_ref].view(np.uint32), own.astype(np.float32).view(np.uint32))
    # in place over the logits
    api.grace_gtm_mask_logits(d_logits, None, dev(score), dev(node), dev(key), trie_s, matcher, d_logits, None, B, M, depth, status)
    assert np.array_equal(d_logits.cpu().numpy().view(np.uint32), h_cand.view(np.uint32))


def test_gtm_mask_flags_nan_and_bad_node(api):
    V, L = 64, 3
    sids, trie, elig, node, key, score, logp = _mask_problem(3, V, L, 500, 1, 8, 1)
    bits, base, _ = api.grace_trie_build_dense(sids, V)
    trie_s = api.make_trie(dev(bits), dev(base), V, L, trie.num_nodes)
    toks, _ = trie.lookup(int(node[0]))
    logp[0, toks[0]] = np.nan
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    cand = torch.empty((8, V), device=DEV)
    api.grace_gtm_mask(dev(logp), dev(score), dev(node), dev(key), trie_s, api.make_matcher(api.MATCH_NONE), cand,
                       None, 1, 8, 1, status)
    assert status.item() & api.DEV_NAN
    status.zero_()
    node2 = node.copy()
    node2[3] = trie.num_nodes + 5
    api.grace_gtm_mask(dev(synth.logp_rows(synth.rng_for(4, 9), 8, V)), dev(score), dev(node2), dev(key), trie_s,
                       api.make_matcher(api.MATCH_NONE), cand, None, 1, 8, 1, status)
    assert status.item() & api.DEV_BAD_INDEX
    assert torch.isneginf(cand[3]).all()


# ------------------------------------------------------------------------------------------
# the paper's index form: CSR child entries + deduplicated per-node rows (Sections 4.2-4.4, 5.4)
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("V,L,n_sids,B,M,depth,n_loc", [
    (64, 3, 2000, 2, 16, 1, 8), (1024, 4, 60000, 3, 37, 1, 64), (1024, 4, 60000, 2, 64, 2, 64),
    (2048, 4, 30000, 2, 9, 0, 64), (1024, 4, 60000, 2, 20, 3, 0),
])
def test_gtm_lookup_paper_form_matches_oracle(api, V, L, n_sids, B, M, depth, n_loc):
    if depth == 0:
        M = 1
    rng = synth.rng_for(4, 500 + V + depth)
    sids = synth.catalog(rng, n_sids, V, L)
    trie = SidTrie(sids, V)
    layout = synth.TargetingLayout()
    loc_rows = synth.location_rows(rng, layout)
    ad_sid, ad_bm, ad_bl = synth.ads_for_sids(rng, n_sids, layout, loc_rows)
    ubm, ubl, _ = synth.request_attributes(rng, B, layout, loc_rows, n_loc=max(n_loc, 1))
    if n_loc == 0:
        ubl = ubl[:, :0]                                         # no location row: nothing may match
    ubm[0] = 0                                                   # a request without attribute constraints
    o_index = OM.NodeMatcherIndex(trie, sids, ad_sid, ad_bm, ad_bl)
    # beams on random catalog prefixes of the given depth (+ a dead one)
    node = np.full(B * M, -1, dtype=np.int32)
    key = np.zeros(B * M, dtype=np.uint64)
    for b in range(B):
        pref = synth.beam_prefixes_from_sids(rng, sids, depth, M) if depth else np.zeros((1, 0), np.int32)
        for i, pr in enumerate(pref):
            node[b * M + i] = trie.walk(pr)
        key[b * M: b * M + pref.shape[0]] = OM.prefix_keys(pref)
    if M > 1:
        node[-1] = -1
    score = np.concatenate([synth.descending_scores(rng, M, max(depth, 1)) for _ in range(B)])
    logp = synth.logp_rows(rng, B * M, V)
    cand_ref, allow_ref, child_ref = OG.gtm_mask(logp, score, node, key, depth, trie,
                                                 OM.NodeRowsMatcher(trie, o_index, ubm, ubl), B, M)
    if n_loc == 0:
        assert not allow_ref.any()
    else:
        assert allow_ref.any() and not allow_ref.all()
    h_index = api.grace_gtm_index_build(sids, V, ad_sid, ad_bm, ad_bl)
    index = api.make_gtm_index(h_index, ubm, np.ascontiguousarray(ubl), DEV)
    cand = torch.full((B * M, V), 7.0, device=DEV)
    allow = torch.zeros((B * M, V // 64), dtype=torch.int64, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    api.grace_gtm_lookup(dev(logp), dev(score), dev(node), index, cand, allow, B, M, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert np.array_equal(host_u64(allow), OG.pack_allow_bits(allow_ref))
    assert np.array_equal(cand.cpu().numpy().view(np.uint32), cand_ref.view(np.uint32))
    # state update through the CSR form
    K = min(32, M * V)
    sc, flat, par, tok = OT.beam_topk(cand_ref.reshape(B, M * V), K, V)
    node_ref, key_ref = OT.update_beam_state(trie, par, tok, sc, node, key, depth, M)
    new_node = torch.empty(B * K, dtype=torch.int32, device=DEV)
    new_key = torch.empty(B * K, dtype=torch.int64, device=DEV)
    api.grace_beam_update_csr(dev(par), dev(tok), dev(sc), dev(node), dev(key), index, new_node, new_key, B, K, M,
                              depth, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert np.array_equal(new_node.cpu().numpy(), node_ref)
    assert np.array_equal(host_u64(new_key), key_ref)


@pytest.mark.parametrize("policy,depth,M", [(("static", [0, 4, 3, 2, 1]), 1, 33), (("static", [0, 4, 3, 2, 1]), 0, 1),
                                            (("dynamic", 0.35, 6), 2, 40), (("dynamic", 0.0, 16), 1, 20)])
def test_gtm_lookup_kway_partitions_match_oracle(api, policy, depth, M):
    """k-way partitioned rows (Section 4.2 "k-way partition"): a child is kept iff ANY of its groups passes the
    bitmask and the Bloom test; the kernel scans the partition slots of the beam's node."""
    from oracle import kway as KW
    V, L, n_sids, B = 256, 4, 6000, 3
    rng = synth.rng_for(4, 700 + depth)
    sids = synth.catalog(rng, n_sids, V, L)
    trie = SidTrie(sids, V)
    layout = synth.TargetingLayout()
    loc_rows = synth.location_rows(rng, layout)
    ad_sid, ad_bm, ad_bl = synth.ads_for_sids(rng, n_sids, layout, loc_rows)
    ubm, ubl, _ = synth.request_attributes(rng, B, layout, loc_rows, n_loc=64)
    ubm[0] = 0
    o_index = KW.KWayMatcherIndex(trie, sids, ad_sid, ad_bm, ad_bl, policy)
    node = np.full(B * M, -1, dtype=np.int32)
    key = np.zeros(B * M, dtype=np.uint64)
    for b in range(B):
        pref = synth.beam_prefixes_from_sids(rng, sids, depth, M) if depth else np.zeros((1, 0), np.int32)
        for i, pr in enumerate(pref):
            node[b * M + i] = trie.walk(pr)
        key[b * M: b * M + pref.shape[0]] = OM.prefix_keys(pref)
    score = np.concatenate([synth.descending_scores(rng, M, max(depth, 1)) for _ in range(B)])
    logp = synth.logp_rows(rng, B * M, V)
    cand_ref, allow_ref, _ = OG.gtm_mask(logp, score, node, key, depth, trie,
                                         KW.KWayRowsMatcher(trie, o_index, ubm, ubl), B, M)
    # partitioning only removes candidates of the union form, and does remove some
    plain_ref = OG.gtm_mask(logp, score, node, key, depth, trie,
                            OM.NodeRowsMatcher(trie, OM.NodeMatcherIndex(trie, sids, ad_sid, ad_bm, ad_bl), ubm, ubl), B, M)[1]
    assert not (allow_ref & ~plain_ref).any() and allow_ref.any()
    if policy[0] == "static":
        h_index = api.grace_gtm_index_build_kway(sids, V, ad_sid, ad_bm, ad_bl, k_level=policy[1])
    else:
        h_index = api.grace_gtm_index_build_kway(sids, V, ad_sid, ad_bm, ad_bl, fill_target=policy[1], k_max=policy[2])
    assert np.array_equal(h_index["part_offsets"], o_index.part_offsets)
    index = api.make_gtm_index(h_index, ubm, np.ascontiguousarray(ubl), DEV)
    cand = torch.full((B * M, V), 7.0, device=DEV)
    allow = torch.zeros((B * M, V // 64), dtype=torch.int64, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    api.grace_gtm_lookup(dev(logp), dev(score), dev(node), index, cand, allow, B, M, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert np.array_equal(host_u64(allow), OG.pack_allow_bits(allow_ref))
    assert np.array_equal(cand.cpu().numpy().view(np.uint32), cand_ref.view(np.uint32))



# ------------------------------------------------------------------------------------------
# beam top-k
# ------------------------------------------------------------------------------------------
def _run_topk(api, cand: np.ndarray, K: int, V: int):
    B, N = cand.shape
    d_cand = dev(cand)
    ws = torch.empty(api.grace_beam_topk_workspace_bytes(B, N, K), dtype=torch.uint8, device=DEV)
    ws.fill_(0xAB)                                           # contents on entry must not matter
    score = torch.empty((B, K), device=DEV)
    flat = torch.empty((B, K), dtype=torch.int32, device=DEV)
    parent = torch.empty_like(flat)
    token = torch.empty_like(flat)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    api.grace_beam_topk(d_cand, K, V, score, flat, parent, token, ws, status)
    torch.cuda.synchronize()
    return score.cpu().numpy(), flat.cpu().numpy(), parent.cpu().numpy(), token.cpu().numpy(), status.item()


def _check_topk(api, cand, K, V, expect_exact_path=None):
    s_ref, f_ref, p_ref, t_ref = OT.beam_topk(cand, K, V)
    s, f, p, t, status = _run_topk(api, cand, K, V)
    assert not (status & (api.DEV_NAN | api.DEV_BAD_INDEX))
    assert np.array_equal(f, f_ref)
    assert np.array_equal(s.view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(p, p_ref) and np.array_equal(t, t_ref)
    if expect_exact_path is not None:
        assert bool(status & api.DEV_TOPK_EXACT_PATH) == expect_exact_path
    return status


@pytest.mark.parametrize("B,M,V,K", [(1, 16, 64, 16), (3, 7, 192, 50), (2, 33, 1024, 2048), (1, 1, 64, 64),
                                     (2, 1, 64, 100), (3, 1, 512, 1024), (1, 3, 64, 1000)])   # beams wider than M * V
def test_topk_small_shapes(api, B, M, V, K):
    rng = synth.rng_for(4, 100 + M)
    cand = synth.normal_f32(rng, (B, M * V), 3.0)
    _check_topk(api, cand, K, V)
    cand[rng.random(cand.shape) < 0.9] = -np.inf                # mostly masked: -inf takes part
    _check_topk(api, cand, K, V)


@pytest.mark.parametrize("B,M,V,K,density", [
    (2, 16, 64, 16, 0.3), (3, 7, 192, 50, 0.05), (2, 300, 1024, 2048, 0.05), (2, 300, 1024, 2048, 0.0005),
    (1, 1, 512, 1024, 0.5),                       # wider than the candidate set
    (2, 2100, 2048, 2048, 0.05), (2, 2100, 2048, 2048, 0.0005), (1, 2048, 2048, 4096, 1.0),   # sampled path, three densities
])
def test_topk_on_candidates_that_are_never_materialised(api, B, M, V, K, density):
    """grace_beam_topk_masked: logits + allow bits + row scores + row log-sum-exp in, the selection of
    grace_beam_topk over score + (logit - lse) / -inf out, bit for bit (including a dead row and an empty request)."""
    rng = synth.rng_for(4, 300 + M + V)
    R = B * M
    logits = synth.normal_f32(rng, (R, V), 1.5)
    lse = (np.log(np.exp(logits.astype(np.float64)).sum(1))).astype(np.float32)
    score = (-np.abs(synth.normal_f32(rng, R, 2.0))).astype(np.float32)
    allow = rng.random((R, V)) < density
    allow[R // 2] = False                                       # a dead beam: nothing allowed, lse irrelevant
    lse[R // 2] = 0.0
    if B > 1 and density < 0.01:
        allow[M:2 * M] = False                                  # a request without a single candidate
    cand = np.where(allow, score[:, None] + (logits - lse[:, None]), np.float32(-np.inf)).astype(np.float32)
    bits = OG.pack_allow_bits(allow)
    s_ref, f_ref, p_ref, t_ref = OT.beam_topk(cand.reshape(B, M * V), K, V)
    ws = torch.empty(api.grace_beam_topk_workspace_bytes(B, M * V, K), dtype=torch.uint8, device=DEV)
    ws.fill_(0xAB)
    sc = torch.empty((B, K), device=DEV)
    fl = torch.empty((B, K), dtype=torch.int32, device=DEV)
    pa, tk = torch.empty_like(fl), torch.empty_like(fl)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    api.grace_beam_topk_masked(dev(logits), dev(bits.view(np.int64)), dev(score), dev(lse), B, M, K, sc, fl, pa, tk, ws, status)
    torch.cuda.synchronize()
    assert not (status.item() & (api.DEV_NAN | api.DEV_BAD_INDEX))
    assert np.array_equal(fl.cpu().numpy(), f_ref)
    assert np.array_equal(sc.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(pa.cpu().numpy(), p_ref) and np.array_equal(tk.cpu().numpy(), t_ref)
    # and identical to the dense entry point on the materialised candidates
    s2, f2, p2, t2, _ = _run_topk(api, cand.reshape(B, M * V), K, V)
    assert np.array_equal(f2, f_ref) and np.array_equal(s2.view(np.uint32), s_ref.view(np.uint32))


def test_topk_sampled_path_dense_and_masked(api):
    """N large enough for the sampled-threshold path: dense scores, then masks of several densities."""
    B, M, V, K = 3, 300, 1024, 2048
    rng = synth.rng_for(4, 200)
    logp = synth.logp_rows(rng, B * M, V)
    score = np.concatenate([synth.descending_scores(rng, M, 2) for _ in range(B)])
    cand = (score[:, None] + logp).astype(np.float32).reshape(B, M * V)
    _check_topk(api, cand, K, V, expect_exact_path=False)
    for density in (0.2, 0.01, 0.005):                          # 0.005 * 307200 = 1536 finite < K: underfull
        masked = cand.copy()
        masked[rng.random(cand.shape) >= density] = -np.inf
        _check_topk(api, masked, K, V, expect_exact_path=False)
    _check_topk(api, cand, 1, V)
    _check_topk(api, cand, 4096, V)


def test_topk_adversarial_inputs_take_the_exact_path_and_stay_exact(api):
    B, N, V, K = 2, 300 * 1024, 1024, 2048
    rng = synth.rng_for(4, 300)
    same = np.full((B, N), -1.5, dtype=np.float32)              # all ties: lowest indices win
    _check_topk(api, same, K, V, expect_exact_path=True)
    ninf = np.full((B, N), -np.inf, dtype=np.float32)           # everything masked
    _check_topk(api, ninf, K, V)
    few = rng.integers(0, 7, size=(B, N)).astype(np.float32)    # 7 distinct values, huge tie groups
    few[0, 5] = -0.0
    _check_topk(api, few, K, V, expect_exact_path=True)
    zeros = np.zeros((B, N), dtype=np.float32)
    zeros[:, ::2] = -0.0                                        # -0.0 == +0.0
    zeros[:, 1000:] = -1.0
    _check_topk(api, zeros, K, V)
    burst = np.full((B, N), -np.inf, dtype=np.float32)          # a dense run of ties above a sparse rest:
    burst[rng.random((B, N)) < 0.003] = -3.0                    # thousands of hits inside one tile of the
    burst[0, :5000] = 0.5                                       # collecting pass, but fewer than the list holds
    burst[1, 70000:73000] = 0.25
    _check_topk(api, burst, 1500, V)
    ramp = np.arange(N, dtype=np.float32)[None].repeat(B, 0)   # sorted ascending: sample is badly stratified
    _check_topk(api, ramp, K, V)
    _check_topk(api, -ramp, K, V)


def test_topk_outliers_clusters_and_tie_groups_on_the_sampled_path(api):
    """Inputs that stress the range histograms of the sampled path: an outlier that stretches the key range of
    the sample (the threshold search has to look closer), tie groups of tens of candidates around the K-th
    value (ranked by index inside a bucket of the counting sort), values clustered on both sides of zero."""
    B, M, V, K = 3, 300, 1024, 2048
    rng = synth.rng_for(4, 302)
    cand = (synth.normal_f32(rng, (B, M * V), 3.0) - 8.0).astype(np.float32)
    wild = cand.copy()
    wild[0, 12345] = 1e30
    wild[1, 777] = np.inf
    wild[2, 5] = 3e38
    wild[2, 4096] = 1e-30
    _check_topk(api, wild, K, V, expect_exact_path=False)
    stepped = (np.round(cand * 64.0) / 64.0).astype(np.float32)
    _check_topk(api, stepped, K, V, expect_exact_path=False)
    _check_topk(api, stepped, 100, V)
    near_zero = (synth.normal_f32(rng, (B, M * V), 1.0) * np.float32(1e-3)).astype(np.float32)
    _check_topk(api, near_zero, K, V)
    near_zero[:, ::3] = 0.0
    near_zero[:, 1::3] = -0.0
    _check_topk(api, near_zero, K, V)


def test_topk_flags_nan(api):
    cand = synth.normal_f32(synth.rng_for(4, 301), (1, 4096))
    cand[0, 77] = np.nan
    *_, status = _run_topk(api, cand, 16, 64)
    assert status & api.DEV_NAN


# ------------------------------------------------------------------------------------------
# beam-state update
# ------------------------------------------------------------------------------------------
def test_beam_update_matches_oracle(api):
    V, L, B, M, K = 1024, 4, 3, 40, 64
    sids, trie, elig, node, key, score, logp = _mask_problem(11, V, L, 60000, B, M, 2)
    bits, base, _ = api.grace_trie_build_dense(sids, V)
    trie_s = api.make_trie(dev(bits), dev(base), V, L, trie.num_nodes)
    cand, _, _ = OG.gtm_mask(logp, score, node, key, 2, trie, OG.NoMatcher(), B, M)
    sc, flat, par, tok = OT.beam_topk(cand.reshape(B, M * V), K, V)       # includes -inf picks (underfull)
    assert np.isneginf(sc).any() and np.isfinite(sc).any()
    node_ref, key_ref = OT.update_beam_state(trie, par, tok, sc, node, key, 2, M)
    new_node = torch.empty(B * K, dtype=torch.int32, device=DEV)
    new_key = torch.empty(B * K, dtype=torch.int64, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    api.grace_beam_update(dev(par), dev(tok), dev(sc), dev(node), dev(key), trie_s, new_node, new_key, B, K, M, 2, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert np.array_equal(new_node.cpu().numpy(), node_ref)
    assert np.array_equal(host_u64(new_key), key_ref)


# ------------------------------------------------------------------------------------------
# self-attention
# ------------------------------------------------------------------------------------------
def _self_attn_problem(seed, B, beam_sizes, H, d, L):
    rng = synth.rng_for(3, seed)
    t = len(beam_sizes) - 1
    R_max = B * max(beam_sizes)
    kc = np.zeros((L, R_max, H, d), dtype=np.uint16)
    vc = np.zeros((L, R_max, H, d), dtype=np.uint16)
    parents = np.zeros((L, R_max), dtype=np.int32)
    for j in range(t):
        n = B * beam_sizes[j]
        kc[j, :n] = synth.normal_bf16(rng, (n, H, d))
        vc[j, :n] = synth.normal_bf16(rng, (n, H, d))
    for j in range(1, t + 1):
        parents[j, :B * beam_sizes[j]] = synth.uniform_parents(rng, B, beam_sizes[j - 1], beam_sizes[j])
    qkv = synth.normal_bf16(rng, (B * beam_sizes[t], 3, H, d))
    return qkv, kc, vc, parents


@pytest.mark.parametrize("B,beam_sizes,H,d", [
    (3, [1], 8, 64), (3, [1, 37], 8, 64), (2, [1, 50, 70], 8, 64), (2, [1, 64, 64, 130], 8, 64),
    (2, [5, 64, 64, 64, 33], 8, 64), (1, [1, 16, 16], 4, 32), (2, [1, 20, 20, 20], 16, 64), (2, [1, 9, 9], 4, 128),
    (1, [2, 3, 4, 5, 6, 7, 8, 9], 2, 64),
    (2, [1, 24, 40, 40], 16, 128),          # the paper's decoder width: rows of 2048 = two 1024-element segments
    (1, [1, 10, 10], 20, 64),               # 1280-wide rows: ragged second segment
    (1, [1, 6, 6], 64, 128),                # the widest row the kernel takes: 8192 elements, eight segments
])
def test_self_attn_matches_oracle(api, B, beam_sizes, H, d):
    L = max(5, len(beam_sizes))
    t = len(beam_sizes) - 1
    qkv, kc, vc, parents = _self_attn_problem(17 * t + H, B, beam_sizes, H, d, L)
    scale = 1.0 / np.sqrt(d)
    par_list = [None] + [parents[j] for j in range(1, t + 1)]
    ref, kc_ref, vc_ref = OA.self_attn(f64(qkv), f64(kc), f64(vc), par_list, beam_sizes, t, B, scale)
    d_kc, d_vc = dev_bf16(kc), dev_bf16(vc)
    R = B * beam_sizes[t]
    out = torch.zeros((R, H, d), dtype=torch.bfloat16, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    api.grace_self_attn(dev_bf16(qkv), d_kc, d_vc, dev(parents), beam_sizes, out, B, t, scale, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert_attention_close(out.float().cpu().numpy(), ref, "self-attn out")
    # cache write: slab t holds exactly the rows' k, v; everything else untouched (bit-exact)
    kc_exp, vc_exp = kc.copy(), vc.copy()
    kc_exp[t, :R], vc_exp[t, :R] = qkv[:, 1], qkv[:, 2]
    assert np.array_equal(d_kc.view(torch.int16).cpu().numpy().view(np.uint16), kc_exp)
    assert np.array_equal(d_vc.view(torch.int16).cpu().numpy().view(np.uint16), vc_exp)


@pytest.mark.parametrize("B,beam_sizes,H,d", [
    (3, [1], 8, 64), (2, [1, 50, 70], 8, 64), (2, [1, 64, 64, 130], 8, 64), (2, [5, 64, 64, 64, 33], 8, 64),
    (1, [1, 16, 16], 4, 32), (2, [1, 24, 40, 40], 16, 128), (1, [1, 10, 10], 20, 64), (1, [1, 6, 6], 64, 128),
    (1, [2, 3, 4, 5, 6, 7, 8, 9], 2, 64),   # the longest prefix the kernel takes (T_self = 8)
])
def test_self_attn_in_place_matches_oracle(api, B, beam_sizes, H, d):
    """The cache held in place: slab j = the QKV projection of step j; the kernel reads the K and V thirds of the
    slabs and writes nothing but its output (the slabs must come back bit for bit)."""
    L = max(5, len(beam_sizes))
    t = len(beam_sizes) - 1
    qkv, kc, vc, parents = _self_attn_problem(17 * t + H, B, beam_sizes, H, d, L)
    scale = 1.0 / np.sqrt(d)
    par_list = [None] + [parents[j] for j in range(1, t + 1)]
    ref, _, _ = OA.self_attn(f64(qkv), f64(kc), f64(vc), par_list, beam_sizes, t, B, scale)
    R_max = kc.shape[1]
    rng = synth.rng_for(3, 991 + t)
    slabs = synth.normal_bf16(rng, (L, R_max, 3, H, d))         # q thirds of older slabs: noise nobody may read
    slabs[:, :, 1], slabs[:, :, 2] = kc, vc
    R = B * beam_sizes[t]
    slabs[t, :R] = qkv
    d_slabs = dev_bf16(slabs)
    out = torch.zeros((R, H, d), dtype=torch.bfloat16, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    api.grace_self_attn_inplace(d_slabs, dev(parents), beam_sizes, out, B, t, scale, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert_attention_close(out.float().cpu().numpy(), ref, "self-attn (in place) out")
    assert np.array_equal(d_slabs.view(torch.int16).cpu().numpy().view(np.uint16), slabs)


def test_self_attn_flags_bad_parent(api):
    B, sizes, H, d = 1, [1, 8], 8, 64
    qkv, kc, vc, parents = _self_attn_problem(5, B, sizes, H, d, 5)
    parents[1, 3] = 99
    out = torch.zeros((8, H, d), dtype=torch.bfloat16, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    api.grace_self_attn(dev_bf16(qkv), dev_bf16(kc), dev_bf16(vc), dev(parents), sizes, out, B, 1, 0.125, status)
    torch.cuda.synchronize()
    assert status.item() & api.DEV_BAD_INDEX


# ------------------------------------------------------------------------------------------
# cross-attention
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("B,M,H,d,T", [
    (1, 16, 4, 32, 64),            # config 1
    (2, 5, 2, 64, 7),              # tiny, ragged
    (2, 130, 8, 64, 128),          # tensor-core shape, ragged M tile
    (3, 256, 8, 64, 512),          # config-2 slice
    (2, 384, 4, 64, 1024),         # long encoder
    (2, 70, 2, 64, 200),           # T not a multiple of the K/V block
    (2, 33, 2, 128, 96),           # head size 128 (two 64-wide halves per tile): one ragged block
    (2, 300, 16, 128, 128),        # the paper's decoder shape: 16 heads of 128, 128 context tokens
    (1, 130, 4, 128, 333),         # head size 128 over several K/V blocks, ragged M and T
    (1, 1, 8, 64, 1024),           # step 0 of the decode loop: one row per request
    (32, 1, 8, 64, 1024),          # the same at the serving batch size (row-per-CTA kernel)
    (2, 3, 4, 128, 200),           # a few rows, head size 128, ragged split of the positions over the warps
    (4, 8, 2, 64, 130),            # the widest beam the row-per-CTA kernel takes
    (3, 2, 4, 64, 5),              # fewer positions than warps
    (2, 1, 2, 64, 1),              # a single encoder position: the softmax is the identity (row-per-CTA kernel)
    (1, 200, 2, 64, 1),            # the same through the tensor-core kernel (one valid column in a 128-wide block)
    (1, 40, 2, 128, 1),
])
def test_cross_attn_matches_oracle(api, B, M, H, d, T):
    rng = synth.rng_for(2, B * 1000 + M + T)
    q = synth.normal_bf16(rng, (B, M, H, d))
    k = synth.normal_bf16(rng, (B, H, T, d))
    v = synth.normal_bf16(rng, (B, H, T, d))
    scale = 1.0 / np.sqrt(d)
    ref, lse_ref = OA.cross_attn(f64(q), f64(k), f64(v), scale)
    out = torch.zeros((B * M, H, d), dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros((B * M, H), dtype=torch.float32, device=DEV)
    api.grace_cross_attn(dev_bf16(q).reshape(B * M, H, d), dev_bf16(k), dev_bf16(v), out, scale, lse)
    torch.cuda.synchronize()
    assert_attention_close(out.float().cpu().numpy().reshape(B, M, H, d), ref, "cross-attn out")
    np.testing.assert_allclose(lse.cpu().numpy().reshape(B, M, H), lse_ref, atol=2e-3, rtol=0)


def test_cross_attn_strided_kv_layout(api):
    """K/V stored [B, T, H, d] (projection output order) are read through strides."""
    B, M, H, d, T = 2, 140, 8, 64, 256
    rng = synth.rng_for(2, 77)
    q = synth.normal_bf16(rng, (B, M, H, d))
    k_bthd = synth.normal_bf16(rng, (B, T, H, d))
    v_bthd = synth.normal_bf16(rng, (B, T, H, d))
    scale = 0.125
    ref, _ = OA.cross_attn(f64(q), f64(k_bthd).transpose(0, 2, 1, 3), f64(v_bthd).transpose(0, 2, 1, 3), scale)
    out = torch.zeros((B * M, H, d), dtype=torch.bfloat16, device=DEV)
    api.grace_cross_attn(dev_bf16(q).reshape(B * M, H, d), dev_bf16(k_bthd).permute(0, 2, 1, 3),
                         dev_bf16(v_bthd).permute(0, 2, 1, 3), out, scale)
    torch.cuda.synchronize()
    assert_attention_close(out.float().cpu().numpy().reshape(B, M, H, d), ref, "cross-attn strided")


@pytest.mark.parametrize("B,M,H,d,T", [(5, 300, 4, 64, 200), (3, 520, 2, 64, 330), (4, 20, 2, 32, 70), (3, 40, 2, 128, 150)])
def test_cross_attn_with_per_request_encoder_lengths(api, B, M, H, d, T):
    """grace_cross_attn_varlen: every request attends to its own number of encoder positions (full, a block
    boundary, one, none, ragged); positions beyond it must have no influence, whatever they hold."""
    rng = synth.rng_for(2, 900 + M + T)
    q = synth.normal_bf16(rng, (B, M, H, d))
    k = synth.normal_bf16(rng, (B, H, T, d))
    v = synth.normal_bf16(rng, (B, H, T, d))
    enc_len = np.array([T, 64, 1, 0, T - 37][:B], dtype=np.int32)
    scale = d ** -0.5
    ref, lse_ref = OA.cross_attn_varlen(f64(q), f64(k), f64(v), enc_len, scale)
    # poison the padding: huge keys and values beyond each request's length
    kf, vf = synth.bf16_bits_to_f32(k).copy(), synth.bf16_bits_to_f32(v).copy()
    for b in range(B):
        kf[b, :, enc_len[b]:] = 50.0
        vf[b, :, enc_len[b]:] = -1000.0
    out = torch.full((B * M, H, d), 7.0, dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros((B * M, H), dtype=torch.float32, device=DEV)
    api.grace_cross_attn_varlen(dev_bf16(q).reshape(B * M, H, d), dev(kf).to(torch.bfloat16), dev(vf).to(torch.bfloat16),
                                out, dev(enc_len), scale, lse)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy().reshape(B, M, H, d)
    assert_attention_close(got, ref, "cross-attn varlen")
    empty = enc_len == 0
    assert (got[empty] == 0).all()
    got_lse = lse.cpu().numpy().reshape(B, M, H)
    assert np.isneginf(got_lse[empty]).all()
    np.testing.assert_allclose(got_lse[~empty], lse_ref[~empty], atol=2e-3, rtol=0)


@pytest.mark.parametrize("B,M,H,d,T", [(2, 300, 2, 64, 640),
                                       # head size 128 (its own kernel and threshold, 2^8), several items per CTA so
                                       # that both output accumulators are rescaled under way
                                       (20, 300, 8, 128, 640)])
def test_cross_attn_with_scores_that_keep_growing(api, B, M, H, d, T):
    """Keys whose scores rise along the encoder positions by far more than the lazy-rescaling threshold
    (2^16 between neighbouring blocks): the running maximum moves in almost every block and the output
    accumulator is rescaled under way; and rows whose maximum sits in the first block, where it never is."""
    rng = synth.rng_for(2, 950 + d)
    q = np.abs(synth.bf16_bits_to_f32(synth.normal_bf16(rng, (B, M, H, d)))) + 0.5     # positive queries
    q[:, ::2] *= -1.0                                                                  # every second row: scores fall instead
    ramp = np.linspace(0.0, 9.0, T, dtype=np.float32)[None, None, :, None]
    k = synth.bf16_bits_to_f32(synth.normal_bf16(rng, (B, H, T, d))) * 0.1 + ramp
    v = synth.bf16_bits_to_f32(synth.normal_bf16(rng, (B, H, T, d)))
    qb, kb, vb = synth.f32_to_bf16_bits(q), synth.f32_to_bf16_bits(k), synth.f32_to_bf16_bits(v)
    scale = 0.125 if d == 64 else 0.125 * 0.5
    ref, _ = OA.cross_attn(f64(qb), f64(kb), f64(vb), scale)
    s_first = (f64(qb)[0, 1, 0] @ f64(kb)[0, 0].T) * scale * np.log2(np.e)
    assert s_first[-1] - s_first[63] > 100.0                    # several thresholds of growth for the rising rows
    out = torch.zeros((B * M, H, d), dtype=torch.bfloat16, device=DEV)
    api.grace_cross_attn(dev_bf16(qb).reshape(B * M, H, d), dev_bf16(kb), dev_bf16(vb), out, scale)
    torch.cuda.synchronize()
    assert_attention_close(out.float().cpu().numpy().reshape(B, M, H, d), ref, "cross-attn growing scores")


# ------------------------------------------------------------------------------------------
# decoder glue
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("M,N,K,relu,res,f32out", [
    (16, 384, 128, False, False, False), (300, 512, 512, False, True, True), (257, 2048, 512, True, False, False),
    (130, 64, 2048, False, True, True), (1, 1536, 512, False, False, False), (100, 80, 64, False, False, True),
    # persistent-kernel shapes (M >= 1024, N >= 256): ragged M and N tiles, every epilogue mode
    (1500, 512, 512, False, True, True), (2125, 1536, 512, False, False, False), (1100, 2048, 512, True, False, False),
    (1300, 512, 2048, False, True, True), (1024, 2048, 512, False, False, True), (1111, 320, 128, False, False, True),
    (40000, 256, 64, True, False, False), (19000, 512, 512, False, True, True),
])
def test_linear_matches_fp64_matmul(api, M, N, K, relu, res, f32out):
    rng = synth.rng_for(5, M + N + K)
    x = synth.normal_bf16(rng, (M, K))
    w = synth.normal_bf16(rng, (N, K), 0.05)
    r = synth.normal_f32(rng, (M, N)) if res else None
    ref = f64(x) @ f64(w).T
    if relu:
        ref = np.maximum(ref, 0)
    if res:
        ref = ref + r
    y = torch.zeros((M, N), dtype=torch.float32 if f32out else torch.bfloat16, device=DEV)
    d_res = None
    if res:
        y.copy_(dev(r))                                           # residual aliases the output
        d_res = y
    api.grace_linear(dev_bf16(x), dev_bf16(w), y, d_res, relu)
    torch.cuda.synchronize()
    got = y.float().cpu().numpy().astype(np.float64)
    abs_sum = np.abs(f64(x)) @ np.abs(f64(w)).T + (np.abs(r) if res else 0.0)
    assert_gemm_close(got, ref, abs_sum, 0 if f32out else 1, f"linear {M}x{N}x{K}")


@pytest.mark.parametrize("M,N,K", [
    (300, 512, 512), (130, 64, 2048), (7, 128, 64),                       # small-tile kernel
    (1500, 512, 512), (1300, 512, 2048), (19000, 512, 512), (1111, 320, 128),   # persistent kernel, ragged tiles
])
def test_linear_add_into_bf16_residual_stream(api, M, N, K):
    rng = synth.rng_for(5, 7 * M + N + K)
    x = synth.normal_bf16(rng, (M, K))
    w = synth.normal_bf16(rng, (N, K), 0.05)
    r = synth.normal_bf16(rng, (M, N))
    ref = f64(x) @ f64(w).T + f64(r)
    y = dev_bf16(r).clone()
    api.grace_linear_add_bf16(dev_bf16(x), dev_bf16(w), y)
    torch.cuda.synchronize()
    got = y.float().cpu().numpy().astype(np.float64)
    # product rounded to bf16 (2^-9 of |x w^T|), then a bf16 add (2^-9 of the sum): the abs-sum term carries
    # the first rounding when product and residual cancel
    abs_sum = np.abs(f64(x)) @ np.abs(f64(w)).T + np.abs(f64(r))
    prod = np.abs(f64(x) @ f64(w).T)
    assert_gemm_close(got, ref + 0.0, abs_sum + 2.0 ** 11 * prod, 1, f"linear_add_bf16 {M}x{N}x{K}")
    err = np.abs(got - ref) / np.maximum(np.abs(ref), np.abs(f64(r)))
    assert np.median(err) <= 2.0 ** -8


def test_layer_norm_embed_bf16_stream(api):
    rng = synth.rng_for(5, 10)
    for R, D in ((77, 512), (5, 128), (33, 1024), (9, 2048), (6, 72)):
        xb = synth.normal_bf16(rng, (R, D), 2.0)
        g, b = synth.normal_f32(rng, D), synth.normal_f32(rng, D)
        out = torch.zeros((R, D), dtype=torch.bfloat16, device=DEV)
        api.grace_layer_norm(dev_bf16(xb), dev(g), dev(b), out, 1e-5)
        x64 = f64(xb)
        ref = (x64 - x64.mean(1, keepdims=True)) / np.sqrt(x64.var(1, keepdims=True) + 1e-5) * g + b
        assert np.abs(out.float().cpu().numpy() - ref).max() <= 2e-2 * max(1, np.abs(ref).max())
    R, D, V = 77, 512, 2048
    emb = synth.normal_bf16(rng, (V + 1, D))
    pos = synth.normal_bf16(rng, (D,))
    tok = rng.integers(0, V + 1, size=R).astype(np.int32)
    xo = torch.zeros((R, D), dtype=torch.bfloat16, device=DEV)
    api.grace_embed(dev(tok), dev_bf16(emb), dev_bf16(pos), xo)
    ref = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(emb)[tok] + synth.bf16_bits_to_f32(pos))
    assert np.array_equal(xo.view(torch.int16).cpu().numpy().view(np.uint16), ref)   # one fp32 add, one RNE rounding


def test_layer_norm_embed_log_softmax(api):
    rng = synth.rng_for(5, 9)
    R, D, V = 77, 512, 2048
    x = synth.normal_f32(rng, (R, D), 2.0) + 0.5
    g, b = synth.normal_f32(rng, D), synth.normal_f32(rng, D)
    out = torch.zeros((R, D), dtype=torch.bfloat16, device=DEV)
    api.grace_layer_norm(dev(x), dev(g), dev(b), out, 1e-5)
    x64 = x.astype(np.float64)
    ref = (x64 - x64.mean(1, keepdims=True)) / np.sqrt(x64.var(1, keepdims=True) + 1e-5) * g + b
    assert np.abs(out.float().cpu().numpy() - ref).max() <= 2e-2 * max(1, np.abs(ref).max())
    emb = synth.normal_bf16(rng, (V + 1, D))
    pos = synth.normal_bf16(rng, (D,))
    tok = rng.integers(0, V + 1, size=R).astype(np.int32)
    xo = torch.zeros((R, D), device=DEV)
    api.grace_embed(dev(tok), dev_bf16(emb), dev_bf16(pos), xo)
    ref = synth.bf16_bits_to_f32(emb)[tok] + synth.bf16_bits_to_f32(pos)
    assert np.array_equal(xo.cpu().numpy(), ref)
    for Vv in (64, 1024, 2048, 4096):
        z = synth.normal_f32(rng, (R, Vv), 3.0)
        d_z = dev(z)
        api.grace_log_softmax(d_z)
        z64 = z.astype(np.float64)
        ref = z64 - z64.max(1, keepdims=True)
        ref = ref - np.log(np.exp(ref).sum(1, keepdims=True))
        np.testing.assert_allclose(d_z.cpu().numpy(), ref, atol=2e-5, rtol=0)


def test_bounded_device_wait_gives_up_and_is_reported(api):
    """A wait on a barrier that nothing completes must end by itself (here after about a millisecond), be
    counted, and leave the context usable: no kernel of this library can hang the GPU on a lost signal."""
    torch.cuda.synchronize()
    api.grace_wait_timeouts()                                   # clear
    assert api.grace_selftest_bounded_wait() == 5               # GRACE_TIMEOUT: the wait gave up as designed
    assert api.grace_wait_timeouts() == 1
    assert api.grace_wait_timeouts() == 0                       # read-and-clear
    # the context is intact: a tensor-core GEMM right after it is still exact to tolerance
    rng = synth.rng_for(5, 4242)
    x, w = synth.normal_bf16(rng, (1100, 256)), synth.normal_bf16(rng, (512, 256), 0.05)
    y = torch.zeros((1100, 512), dtype=torch.bfloat16, device=DEV)
    api.grace_linear(dev_bf16(x), dev_bf16(w), y, None, False)
    torch.cuda.synchronize()
    ref = f64(x) @ f64(w).T
    assert np.abs(y.float().cpu().numpy() - ref).max() <= 2e-2 * max(1.0, np.abs(ref).max())
    assert api.grace_wait_timeouts() == 0


@pytest.mark.parametrize("M,N,K", [(1024, 256, 64), (1500, 2048, 512), (2100, 512, 2048), (33000, 2048, 512)])
def test_logits_gemm_leaves_log_sum_exp_partials(api, M, N, K):
    """grace_linear_f32_lse: the same fp32 product as grace_linear, plus per row and 256-column tile the pair
    (maximum, sum of e^(y - maximum)); merged, they are the row's log-sum-exp."""
    rng = synth.rng_for(5, 13 * M + N + K)
    x = synth.normal_bf16(rng, (M, K))
    w = synth.normal_bf16(rng, (N, K), 0.08)
    y0 = torch.zeros((M, N), dtype=torch.float32, device=DEV)
    api.grace_linear(dev_bf16(x), dev_bf16(w), y0, None, False)
    y = torch.zeros_like(y0)
    part = torch.full((M, N // 256, 2), 7.0, device=DEV)
    api.grace_linear_f32_lse(dev_bf16(x), dev_bf16(w), y, part)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int32), y0.view(torch.int32))
    p = part.cpu().numpy().astype(np.float64)
    yt = y.cpu().numpy().astype(np.float64).reshape(M, N // 256, 256)
    assert np.array_equal(p[:, :, 0], yt.max(2))                                        # the tile maximum, exactly
    np.testing.assert_allclose(p[:, :, 1], np.exp(yt - yt.max(2, keepdims=True)).sum(2), rtol=2e-6)
    lse = p[:, :, 0].max(1) + np.log((p[:, :, 1] * np.exp(p[:, :, 0] - p[:, :, 0].max(1, keepdims=True))).sum(1))
    ref = np.log(np.exp(yt.reshape(M, N) - yt.max((1, 2))[:, None]).sum(1)) + yt.max((1, 2))
    np.testing.assert_allclose(lse, ref, atol=1e-5, rtol=0)
    with pytest.raises(api.GraceError):                                                 # small problems: not offered
        api.grace_linear_f32_lse(dev_bf16(x[:100]), dev_bf16(w), y[:100], part[:100])


@pytest.mark.parametrize("kind,M", [("bloom", 600), ("node", 37)])
def test_mask_kernel_merges_log_sum_exp_partials(api, kind, M):
    """grace_gtm_mask_logits_parts against grace_gtm_mask_logits on the same logits: identical allow bits, the same
    log-sum-exp to fp32 rounding, candidates equal to score + (logit - its own lse)."""
    V, L, B, n_sids, depth = 1024, 4, 2, 60000, 1
    sids, trie, elig, node, key, score, _ = _mask_problem(5 * V + depth + M, V, L, n_sids, B, M, depth)
    rng = synth.rng_for(4, 950 + M)
    logits = synth.normal_f32(rng, (B * M, V), 2.0)
    bits, base, level_start = api.grace_trie_build_dense(sids, V)
    d_bits, d_base = dev(bits), dev(base)
    trie_s = api.make_trie(d_bits, d_base, V, L, trie.num_nodes)
    if kind == "node":
        keep = dev(np.stack([api.grace_node_bitmask_build(sids, V, e, trie.num_nodes) for e in elig]))
        matcher = api.make_matcher(api.MATCH_NODE_BITMASK, keep)
    else:
        keep = dev(np.stack([api.grace_bloom_build(sids, V, e, 14, 4) for e in elig]))
        matcher = api.make_matcher(api.MATCH_PREFIX_BLOOM, keep, 14, 4)
    R, W = B * M, V // 64
    # partials as the GEMM writes them, made here from the logits themselves
    lt = logits.astype(np.float64).reshape(R, V // 256, 256)
    part = np.stack([lt.max(2), np.exp(lt - lt.max(2, keepdims=True)).sum(2)], axis=2).astype(np.float32)
    out = {}
    for name in ("stream", "parts"):
        cand = torch.full((R, V), 3.0, device=DEV)
        allow = torch.zeros((R, W), dtype=torch.int64, device=DEV)
        lse = torch.zeros(R, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        if name == "stream":
            api.grace_gtm_mask_logits(dev(logits), lse, dev(score), dev(node), dev(key), trie_s, matcher, cand, allow, B, M, depth, status)
        else:
            api.grace_gtm_mask_logits_parts(dev(logits), lse, dev(score), dev(node), dev(key), trie_s, matcher, cand, allow, B, M,
                                            depth, dev(part), status)
        torch.cuda.synchronize()
        assert status.item() == 0
        out[name] = (cand.cpu().numpy(), host_u64(allow), lse.cpu().numpy())
    assert np.array_equal(out["stream"][1], out["parts"][1]) and out["parts"][1].any()
    np.testing.assert_allclose(out["parts"][2], out["stream"][2], atol=2e-5, rtol=0)
    live = node >= 0
    cand, lse = out["parts"][0], out["parts"][2]
    allowed = np.isfinite(cand)
    want = (score[:, None] + (logits - lse[:, None])).astype(np.float32)
    assert np.array_equal(cand[allowed].view(np.uint32), want[allowed].view(np.uint32))
    assert not allowed[~live].any()


@pytest.mark.parametrize("M,N,K,relu,f32out", [(300, 384, 128, False, False), (130, 2048, 512, True, False),
                                               (2100, 1536, 512, False, False), (1500, 2048, 512, True, False),
                                               (1100, 512, 512, False, True), (33000, 2048, 512, False, True),
                                               # ragged last column tile in the pair kernel (clamped vector fetches)
                                               (1500, 784, 512, True, False), (1300, 336, 512, False, True),
                                               # one-kernel form of grace_linear_layer_norm (centred, N <= 512), bf16 out
                                               (33000, 512, 512, True, False), (2100, 384, 512, False, False)])
@pytest.mark.parametrize("centred", [False, True])
def test_layer_norm_folded_into_the_gemm(api, M, N, K, relu, f32out, centred):
    """grace_row_stats_bf16 + grace_linear_folded_ln against LayerNorm(x) @ w^T in fp64: the GEMM reads the raw
    bf16 stream, its weights carry the gain, the epilogue applies (rstd, -rstd * mean) and the column vectors.
    centred: the rows of x have zero mean (up to their bf16 rounding) and no column sums are passed."""
    rng = synth.rng_for(5, 17 * M + N + K)
    x = synth.normal_bf16(rng, (M, K), 1.5)
    if centred:
        xc = synth.bf16_bits_to_f32(x).astype(np.float64)
        x = synth.f32_to_bf16_bits((xc - xc.mean(1, keepdims=True)).astype(np.float32))
    else:                                   # a mean the column-sum term has to carry
        x = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(x) + np.float32(0.75))
    x64 = f64(x) + 0.0
    w = synth.normal_bf16(rng, (N, K), 0.05)
    g = (synth.normal_f32(rng, K) * 0.2 + 1.0).astype(np.float32)
    b = (synth.normal_f32(rng, K) * 0.3).astype(np.float32)
    ln = (x64 - x64.mean(1, keepdims=True)) / np.sqrt(x64.var(1, keepdims=True) + 1e-5) * g + b
    ref = ln @ f64(w).T
    if relu:
        ref = np.maximum(ref, 0)
    wf_bits = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(w) * g[None, :])
    cs = f64(wf_bits).sum(1).astype(np.float32)
    cb = (f64(w) @ b.astype(np.float64)).astype(np.float32)
    aff = torch.zeros((M, 2), device=DEV)
    api.grace_row_stats_bf16(dev_bf16(x), aff, 1e-5)
    torch.cuda.synchronize()
    a = aff.cpu().numpy().astype(np.float64)
    rstd = 1.0 / np.sqrt(x64.var(1) + 1e-5)
    np.testing.assert_allclose(a[:, 0], rstd, rtol=2e-6)
    np.testing.assert_allclose(a[:, 1], -rstd * x64.mean(1), rtol=0, atol=2e-6 * (1 + np.abs(rstd * x64.mean(1)).max()))
    y = torch.zeros((M, N), dtype=torch.float32 if f32out else torch.bfloat16, device=DEV)
    part = torch.zeros((M, N // 256, 2), device=DEV) if (f32out and M >= 1024 and N % 256 == 0) else None
    api.grace_linear_folded_ln(dev_bf16(x), dev_bf16(wf_bits), aff, None if centred else dev(cs), dev(cb), y, relu, part)
    torch.cuda.synchronize()
    got = y.float().cpu().numpy().astype(np.float64)
    # folding rounds w * gamma to bf16 once (2^-9 relative per weight, averaging out over K terms)
    tol = 1.2e-2 if f32out else 2e-2
    assert np.abs(got - ref).max() <= tol * max(1.0, np.abs(ref).max()), np.abs(got - ref).max()
    assert np.sqrt(((got - ref) ** 2).sum() / (ref ** 2).sum()) <= 5e-3
    if part is not None:
        p = part.cpu().numpy().astype(np.float64)
        lse = p[:, :, 0].max(1) + np.log((p[:, :, 1] * np.exp(p[:, :, 0] - p[:, :, 0].max(1, keepdims=True))).sum(1))
        want = np.log(np.exp(got - got.max(1, keepdims=True)).sum(1)) + got.max(1)
        np.testing.assert_allclose(lse, want, atol=1e-5, rtol=0)
    # the same as ONE call (for large centred problems one kernel: statistics from the GEMM's own operand tiles)
    y1 = torch.zeros_like(y)
    part1 = torch.zeros_like(part) if part is not None else None
    scratch = torch.full((M, 2), 7.0, device=DEV)
    api.grace_linear_layer_norm(dev_bf16(x), dev_bf16(wf_bits), 1e-5, scratch, None if centred else dev(cs), dev(cb), y1,
                                relu, part1)
    torch.cuda.synchronize()
    got1 = y1.float().cpu().numpy().astype(np.float64)
    assert np.abs(got1 - ref).max() <= tol * max(1.0, np.abs(ref).max()), np.abs(got1 - ref).max()
    assert np.sqrt(((got1 - ref) ** 2).sum() / (ref ** 2).sum()) <= 5e-3
    # against the two-kernel form: the statistics agree to rounding (2e-6), so the outputs do to that times |y|
    # plus, for bf16 outputs, a rounding that may fall the other way
    slack = 1e-5 * np.abs(got) + (0 if f32out else 2.0 ** -7 * np.abs(got)) + 1e-6
    assert (np.abs(got1 - got) <= slack).all(), np.abs(got1 - got).max()
    if part1 is not None:
        np.testing.assert_allclose(part1.cpu().numpy(), part.cpu().numpy(), rtol=2e-5, atol=2e-5)
    in_kernel = centred and M >= 1024 and 256 <= N <= 512 and part is None
    assert bool((scratch == 7.0).all().item()) == in_kernel       # the scratch is touched only by the two-kernel form


@pytest.mark.parametrize("M,N,K,density,folded", [(2100, 2048, 512, 0.2, True), (1100, 512, 512, 0.002, False),
                                                  (1500, 1024, 256, 1.0, True), (1030, 256, 128, 0.0, False),
                                                  (33000, 2048, 512, 0.0005, True)])
def test_logits_gemm_stores_only_the_allowed_logits(api, M, N, K, density, folded):
    """grace_linear_logits_allowed against the dense logits GEMM (grace_linear_f32_lse, or the folded-LayerNorm
    form with partials): where a bit is set the stored value is the dense one bit for bit, everything else keeps
    what the buffer held (or, next to an allowed column, holds the dense value too), and the log-sum-exp partials
    (over ALL columns) are the same bits."""
    rng = synth.rng_for(5, 900 + M + N)
    x = synth.normal_bf16(rng, (M, K), 1.5)
    xc = synth.bf16_bits_to_f32(x).astype(np.float64)
    x = synth.f32_to_bf16_bits((xc - xc.mean(1, keepdims=True)).astype(np.float32))       # centred rows (no col_sum)
    w = synth.normal_bf16(rng, (N, K), 0.05)
    cb = synth.normal_f32(rng, N) if folded else None
    allow = rng.random((M, N)) < density
    allow[M // 2] = True                                     # a full row and an empty one whatever the density
    allow[M // 3] = False
    bits = OG.pack_allow_bits(allow)
    dense = torch.zeros((M, N), device=DEV)
    part = torch.zeros((M, N // 256, 2), device=DEV)
    aff = torch.zeros((M, 2), device=DEV)
    if folded:
        api.grace_linear_layer_norm(dev_bf16(x), dev_bf16(w), 1e-5, aff, None, dev(cb), dense, False, part)
    else:
        api.grace_linear_f32_lse(dev_bf16(x), dev_bf16(w), dense, part)
    sentinel = np.float32(-123.25)
    y = torch.full((M, N), float(sentinel), device=DEV)
    part1 = torch.zeros_like(part)
    api.grace_linear_logits_allowed(dev_bf16(x), dev_bf16(w), dev(bits.view(np.int64)), y, part1, 1e-5,
                                    aff if folded else None, None, dev(cb) if folded else None)
    torch.cuda.synchronize()
    got, ref = y.cpu().numpy(), dense.cpu().numpy()
    assert np.array_equal(got[allow].view(np.uint32), ref[allow].view(np.uint32))
    # elsewhere: what the buffer held, or (columns sharing a 32-byte sector with an allowed one) the dense value
    other = got[~allow]
    assert ((other == sentinel) | (other.view(np.uint32) == ref[~allow].view(np.uint32))).all()
    if density < 0.01:
        assert (other == sentinel).mean() > 0.9
    assert np.array_equal(part1.cpu().numpy().view(np.uint32), part.cpu().numpy().view(np.uint32))
    if folded:                                   # eps < 0: the statistics are the caller's (same kernel, same bits)
        api.grace_row_stats_bf16(dev_bf16(x), aff, 1e-5)
        y2 = torch.full((M, N), float(sentinel), device=DEV)
        api.grace_linear_logits_allowed(dev_bf16(x), dev_bf16(w), dev(bits.view(np.int64)), y2, part1, -1.0, aff, None, dev(cb))
        torch.cuda.synchronize()
        assert torch.equal(y2.view(torch.int32), y.view(torch.int32))


def test_allow_bits_before_the_logits_and_the_merge_of_their_partials(api):
    """grace_gtm_allow_bits leaves the bits the mask kernels leave (and the oracle's mask), from the beam state
    alone; grace_row_lse_from_parts gives the rows' log-sum-exp the mask kernel gives from the same partials, bit
    for bit, 0 on dead rows."""
    V, L, B, M = 1024, 4, 3, 400
    sids, trie, elig, node, key, score, logp = _mask_problem(12, V, L, 60000, B, M, 1)
    node = node.copy()
    node[5] = -1                                             # a dead row
    bits, base, _ = api.grace_trie_build_dense(sids, V)
    trie_s = api.make_trie(dev(bits), dev(base), V, L, trie.num_nodes)
    for kind in ("bloom", "node"):
        if kind == "bloom":
            om = OG.PrefixBloomMatcher([OM.build_prefix_bloom(sids, e, 16, 3) for e in elig])
            keep = dev(np.stack([api.grace_bloom_build(sids, V, e, 16, 3) for e in elig]))
            matcher = api.make_matcher(api.MATCH_PREFIX_BLOOM, keep, 16, 3)
        else:
            om = OG.NodeBitmaskMatcher(np.stack([OM.node_eligibility(trie, sids, e) for e in elig]))
            keep = dev(np.stack([api.grace_node_bitmask_build(sids, V, e, trie.num_nodes) for e in elig]))
            matcher = api.make_matcher(api.MATCH_NODE_BITMASK, keep)
        R = B * M
        logits = (logp * 3.0).astype(np.float32)
        d_logits = dev(logits)
        part = torch.zeros((R, V // 256, 2), device=DEV)
        lg = logits.reshape(R, V // 256, 256).astype(np.float64)
        mx = lg.max(2)
        part.copy_(dev(np.stack([mx, np.exp(lg - mx[:, :, None]).sum(2)], axis=2).astype(np.float32)))
        lse_a, allow_a = torch.zeros(R, device=DEV), torch.zeros((R, V // 64), dtype=torch.int64, device=DEV)
        api.grace_gtm_mask_logits_parts(d_logits, lse_a, dev(score), dev(node), dev(key), trie_s, matcher, None, allow_a,
                                        B, M, 1, part)
        lse_b, allow_b = torch.full((R,), 9.0, device=DEV), torch.full((R, V // 64), -1, dtype=torch.int64, device=DEV)
        api.grace_gtm_allow_bits(dev(node), dev(key), trie_s, matcher, allow_b, B, M, 1)
        api.grace_row_lse_from_parts(part, dev(node), trie_s, lse_b)
        torch.cuda.synchronize()
        assert torch.equal(allow_a, allow_b)
        assert torch.equal(lse_a.view(torch.int32), lse_b.view(torch.int32))
        assert lse_b[5].item() == 0.0
        _, a_ref, _ = OG.gtm_mask(logp, score, node, key, 1, trie, om, B, M)
        assert np.array_equal(allow_b.cpu().numpy().view(np.uint64), OG.pack_allow_bits(a_ref))
    # other numbers of partials per row (the merge kernel packs 4, 2 or 1 rows into a warp): against the definition
    rng = synth.rng_for(4, 1201)
    for n_parts in (1, 2, 8, 12, 16, 17, 32):
        R = B * M
        mx = synth.normal_f32(rng, (R, n_parts), 4.0)
        sm = (1.0 + rng.random((R, n_parts)) * 255.0).astype(np.float32)
        part = dev(np.stack([mx, sm], axis=2).astype(np.float32))
        out = torch.full((R,), 9.0, device=DEV)
        api.grace_row_lse_from_parts(part, dev(node), trie_s, out)
        torch.cuda.synchronize()
        m64 = mx.astype(np.float64)
        want = m64.max(1) + np.log((sm.astype(np.float64) * np.exp(m64 - m64.max(1, keepdims=True))).sum(1))
        want[node < 0] = 0.0
        leaf = node >= trie.num_internal_nodes()
        np.testing.assert_allclose(out.cpu().numpy()[~leaf], want[~leaf], rtol=0, atol=2e-5)


def test_l2_residency_window_is_a_hint_only(api):
    """grace_stream_l2_persist changes where lines live, never what a kernel computes: the same GEMM into the
    same residual stream gives the same bits with the window set, with it cleared, and on another stream."""
    rng = synth.rng_for(5, 4242)
    M, N, K = 4096, 512, 512
    x, w = dev_bf16(synth.normal_bf16(rng, (M, K))), dev_bf16(synth.normal_bf16(rng, (N, K), 0.05))
    base = dev_bf16(synth.normal_bf16(rng, (M, N)))
    outs = []
    for mode in ("plain", "window", "cleared"):
        y = base.clone()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            if mode == "window":
                api.grace_stream_l2_persist(y, 0.5)
            elif mode == "cleared":
                api.grace_stream_l2_persist(y, 1.0)
                api.grace_stream_l2_persist(None)
            api.grace_linear_add_bf16(x, w, y)
        side.synchronize()
        outs.append(y)
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])
    with pytest.raises(Exception):
        api.grace_stream_l2_persist(base, 0.0)
    with pytest.raises(Exception):
        api.grace_stream_l2_persist(base, 1.5)


_DSMEM_CHILD = r"""
import sys, numpy as np, torch
sys.path.insert(0, sys.argv[1])
sys.path.insert(0, sys.argv[1] + "/tests")
import synth
from paper_2608_00938_b200 import api
from test_gpu_ops import _mask_problem
from gpu_util import dev
V, L, B, M = 1024, 4, 2, 600
sids, trie, elig, node, key, score, logp = _mask_problem(13, V, L, 60000, B, M, 1)
bits, base, _ = api.grace_trie_build_dense(sids, V)
trie_s = api.make_trie(dev(bits), dev(base), V, L, trie.num_nodes)
keep = dev(np.stack([api.grace_bloom_build(sids, V, e, 16, 4) for e in elig]))
matcher = api.make_matcher(api.MATCH_PREFIX_BLOOM, keep, 16, 4)
allow = torch.zeros((B * M, V // 64), dtype=torch.int64, device="cuda:0")
api.grace_gtm_allow_bits(dev(node), dev(key), trie_s, matcher, allow, B, M, 1)
torch.cuda.synchronize()
np.save(sys.argv[2], allow.cpu().numpy())
"""


def test_bloom_filter_in_cluster_shared_memory_gives_the_same_bits(api, tmp_path):
    """The variant of grace_gtm_allow_bits that keeps each request's Bloom filter in the shared memory of a
    four-CTA cluster (off by default: measured slower; GRACE_BLOOM_DSMEM selects it) leaves the same allow bits as
    the default form.  The switch is read once per process, so each form runs in a process of its own."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    outs = []
    for flag in (None, "1"):
        env = dict(os.environ)
        env.pop("GRACE_BLOOM_DSMEM", None)
        if flag:
            env["GRACE_BLOOM_DSMEM"] = flag
        out = str(tmp_path / f"allow_{flag}.npy")
        subprocess.run([sys.executable, "-c", _DSMEM_CHILD, root, out], check=True, env=env, timeout=600)
        outs.append(np.load(out))
    assert outs[0].any() and np.array_equal(outs[0], outs[1])
