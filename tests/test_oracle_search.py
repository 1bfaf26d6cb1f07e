"""Pins for oracle.gtm, oracle.topk and oracle.decoder: brute force over all
(row, token) pairs, python sorted(), exhaustive SID enumeration on tiny
catalogs, and the invariants the method guarantees.  CPU only."""
import itertools

import numpy as np
import pytest

import synth
from oracle import decoder as D
from oracle import gtm as G
from oracle import matchers as Mx
from oracle import topk as T
from oracle.sid_trie import SidTrie


def _tiny(seed, V=64, L=3, n=300, frac=0.3, B=2):
    rng = synth.rng_for(1, seed)
    sids = synth.catalog(rng, n, V, L)
    trie = SidTrie(sids, V)
    elig = [synth.eligible_subset(rng, n, frac) for _ in range(B)]
    return rng, sids, trie, elig


@pytest.mark.parametrize("kind", ["none", "node", "bloom"])
def test_gtm_mask_equals_brute_force(kind):
    rng, sids, trie, elig = _tiny(20)
    V, L, B, M, t = 64, 3, 2, 6, 1
    catalog_prefixes = {tuple(s[:l]) for s in sids.tolist() for l in range(L + 1)}
    if kind == "none":
        matcher = G.NoMatcher()
        passes = lambda b, p: True
    elif kind == "node":
        matcher = G.NodeBitmaskMatcher(np.stack([Mx.node_eligibility(trie, sids, e) for e in elig]))
        good = [{tuple(s[:l]) for s, e in zip(sids.tolist(), el) if e for l in range(L + 1)} for el in elig]
        passes = lambda b, p: p in good[b]
    else:
        blooms = [Mx.build_prefix_bloom(sids, e, 12, 4) for e in elig]
        matcher = G.PrefixBloomMatcher(blooms)
        passes = lambda b, p: bool(blooms[b].contains(np.array([Mx.prefix_key(p)]))[0])
    # beams: level-1 prefixes, one dead row per request
    level1 = trie.prefixes[1][:, 0]
    beam_tok = rng.choice(level1, size=(B, M), replace=True)
    node = np.array([trie.walk([x]) for x in beam_tok.reshape(-1)], dtype=np.int32)
    node[M - 1] = -1
    key = Mx.prefix_keys(beam_tok.reshape(-1, 1))
    score = -np.abs(synth.normal_f32(rng, B * M))
    logp = synth.logp_rows(rng, B * M, V)
    cand, allow, child = G.gtm_mask(logp, score, node, key, t, trie, matcher, B, M)
    for r in range(B * M):
        for v in range(V):
            p = (int(beam_tok.reshape(-1)[r]), v)
            want = node[r] >= 0 and p in catalog_prefixes and passes(r // M, p)
            assert allow[r, v] == want
            if want:
                assert cand[r, v] == np.float32(score[r]) + np.float32(logp[r, v])
                assert child[r, v] == trie.walk(p)
            else:
                assert cand[r, v] == -np.inf and child[r, v] == -1
    assert np.array_equal(np.isfinite(cand), allow)
    assert not allow[M - 1].any()
    if kind == "bloom":      # Bloom never drops a truly eligible prefix
        exact = G.gtm_mask(logp, score, node, key, t, trie,
                           G.NodeBitmaskMatcher(np.stack([Mx.node_eligibility(trie, sids, e) for e in elig])), B, M)[1]
        assert not (exact & ~allow).any()
    bits = G.pack_allow_bits(allow)
    for r in range(B * M):
        for v in range(V):
            assert ((int(bits[r, v // 64]) >> (v % 64)) & 1) == int(allow[r, v])


def test_topk_equals_python_sorted():
    rng = np.random.default_rng(4)
    B, M, V, K = 3, 5, 64, 37
    cand = rng.standard_normal((B, M * V)).astype(np.float32)
    cand[rng.random((B, M * V)) < 0.5] = -np.inf
    cand[0, :40] = np.float32(100.0)                     # a run of exact ties at the top
    cand[1, 7], cand[1, 3] = np.float32(-0.0), np.float32(0.0)
    cand[1, cand[1] > 0] = -np.inf                       # make the zeros the top of request 1
    cand[2, 10:] = -np.inf                               # fewer finite than K
    score, flat, parent, token = T.beam_topk(cand, K, V)
    for b in range(B):
        order = sorted(range(M * V), key=lambda i: (-float(cand[b, i]), i))[:K]
        assert flat[b].tolist() == order
        assert np.array_equal(score[b], cand[b, order])
        assert parent[b].tolist() == [i // V for i in order] and token[b].tolist() == [i % V for i in order]
        assert len(set(flat[b].tolist())) == K
        rest = np.delete(cand[b], flat[b])
        assert rest.size == 0 or score[b, -1] >= rest.max()
    assert flat[0].tolist() == list(range(K))
    assert flat[1, :2].tolist() == [3, 7]                # -0.0 ties with +0.0, index decides
    assert np.isneginf(score[2, 10:]).all() and (np.diff(flat[2, 10:]) > 0).all()
    same = T.beam_topk(np.full((1, 200), -1.5, np.float32), 9, 50)
    assert same[1][0].tolist() == list(range(9))
    with pytest.raises(AssertionError):
        T.beam_topk(np.array([[np.nan, 1.0]], np.float32), 1, 2)
    # a beam wider than the candidate set: every candidate in order, then dead entries on candidate 0
    small = np.array([[0.5, -np.inf, 2.0, 0.5, -1.0, -np.inf]], np.float32)
    sc, fl, pa, tk = T.beam_topk(small, 9, 3)
    assert fl[0].tolist() == [2, 0, 3, 4, 1, 5, 0, 0, 0]
    assert sc[0, :4].tolist() == [2.0, 0.5, 0.5, -1.0] and np.isneginf(sc[0, 4:]).all()
    assert pa[0, 6:].tolist() == [0, 0, 0] and tk[0, 6:].tolist() == [0, 0, 0]


def _exhaustive(weights, shp, enc, trie, sids, passes):
    """Score every catalog SID whose prefixes all pass, by running the decoder
    along its own path with a beam of one (no search)."""
    results = []
    ckv = D.cross_kv(weights, shp, enc)
    for sid in sids.tolist():
        if not all(passes(tuple(sid[:l])) for l in range(1, shp.L + 1)):
            continue
        state = D.DecoderState(shp, 1, [1] * shp.L)
        tok, total = shp.V, np.float32(0.0)
        for t in range(shp.L):
            if t > 0:
                state.parents[t] = np.zeros(1, dtype=np.int32)
            logp = D.decoder_forward(weights, shp, state, ckv, np.array([tok]), t, 1).astype(np.float32)
            total = np.float32(total + logp[0, sid[t]])
            tok = sid[t]
        results.append((float(total), tuple(sid)))
    return results


@pytest.mark.parametrize("kind", ["node", "bloom"])
def test_beam_search_is_exhaustive_when_beams_are_wide_enough(kind):
    V, L, n = 64, 3, 40
    rng = synth.rng_for(1, 30)
    sids = synth.catalog(rng, n, V, L)
    trie = SidTrie(sids, V)
    elig = synth.eligible_subset(rng, n, 0.5)
    shp = synth.DecoderShape(2, 32, 2, 16, 64, 32, V, L)
    w = synth.decoder_weights(rng, shp, std=0.3, as_bf16=False)     # larger std: well separated scores
    enc = synth.normal_f32(rng, (1, 5, 32))
    if kind == "node":
        marks = Mx.node_eligibility(trie, sids, elig)
        matcher = G.NodeBitmaskMatcher(marks[None])
        passes = lambda p: bool(marks[trie.walk(p)])
    else:
        bloom = Mx.build_prefix_bloom(sids, elig, 10, 4)            # small filter: real false positives
        matcher = G.PrefixBloomMatcher([bloom])
        passes = lambda p: bool(bloom.contains(np.array([Mx.prefix_key(p)]))[0])
    record = []
    out = D.beam_search(w, shp, enc, trie, matcher, (1, 64, 64), 64, record=record)
    truth = sorted(_exhaustive(w, shp, enc, trie, sids, passes), key=lambda x: -x[0])
    n_valid = int(out["valid"][0].sum())
    assert n_valid == len(truth) and n_valid >= int(elig.sum())
    got = [tuple(s) for s in out["sids"][0, :n_valid].tolist()]
    assert got == [s for _, s in truth]
    np.testing.assert_allclose(out["score"][0, :n_valid], [x for x, _ in truth], rtol=0, atol=2e-5)
    # invariants of Sections 3.1 / 3.2 / 4.1
    catalog = {tuple(s) for s in sids.tolist()}
    assert all(s in catalog for s in got)                                    # CD: catalog-valid
    assert all(passes(s[:l]) for s in got for l in range(1, L + 1))          # GTM: every prefix passes
    for step in record:
        sc = step["out_score"]
        assert (sc[:, 1:] <= sc[:, :-1]).all()                               # sorted within a beam
        par_score = step["score"].reshape(1, -1)[0][step["out_parent"][0]]
        live = ~np.isneginf(sc[0])
        assert (sc[0][live] <= par_score[live]).all()                        # child = parent + logp <= parent
        np.testing.assert_allclose(np.exp(step["logp"].astype(np.float64)).sum(axis=1), 1.0, atol=1e-5)
    assert (~np.isneginf(record[0]["out_score"])).sum() <= V                 # at most |V| prefixes after step 0
    # a schedule wider than the codebook at step 0 (the paper's fixed schedule has this shape) only adds dead beams
    wide = D.beam_search(w, shp, enc, trie, matcher, (1, 100, 100), 100)
    assert int(wide["valid"][0].sum()) == n_valid
    assert [tuple(s_) for s_ in wide["sids"][0, :n_valid].tolist()] == got
    assert np.array_equal(wide["score"][0, :n_valid], out["score"][0, :n_valid])
    dead = record[-1]["new_node"] < 0
    assert np.array_equal(dead, np.isneginf(record[-1]["out_score"].reshape(-1)))


def test_narrow_beam_keeps_the_invariants_and_config1_shape():
    rng = synth.rng_for(1)
    V, L = 64, 3
    sids = synth.catalog(rng, 2000, V, L)
    trie = SidTrie(sids, V)
    elig = synth.eligible_subset(rng, 2000, 0.3)
    marks = Mx.node_eligibility(trie, sids, elig)
    shp = synth.DecoderShape(2, 128, 4, 32, 512, 128, V, L)
    w = synth.decoder_weights(rng, shp, as_bf16=False)
    enc = synth.normal_f32(rng, (1, 64, 128))
    rec64, rec32 = [], []
    out = D.beam_search(w, shp, enc, trie, G.NodeBitmaskMatcher(marks[None]), (1, 16, 16), 16, record=rec64)
    out32 = D.beam_search(w, shp, enc, trie, G.NodeBitmaskMatcher(marks[None]), (1, 16, 16), 16,
                          dtype=np.float32, record=rec32)
    good = {tuple(s) for s, e in zip(sids.tolist(), elig) if e}
    assert out["valid"].all()
    assert all(tuple(s) in good for s in out["sids"][0].tolist())
    assert (np.diff(out["score"][0]) <= 0).all()
    # fp32 and fp64 decoders agree (self-consistency of the unpinned layer internals)
    for a, b in zip(rec64, rec32):
        if np.array_equal(a["tokens"], b["tokens"]):
            np.testing.assert_allclose(a["logp"], b["logp"], atol=1e-5)
    np.testing.assert_allclose(rec64[0]["logp"], rec32[0]["logp"], atol=1e-5)


def test_layer_norm_and_log_softmax_moments():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((7, 33)) * 5 + 2
    y = D.layer_norm(x, np.ones(33), np.zeros(33), eps=0.0)
    np.testing.assert_allclose(y.mean(axis=1), 0, atol=1e-12)
    np.testing.assert_allclose(y.var(axis=1), 1, atol=1e-12)
    g, b = rng.standard_normal(33), rng.standard_normal(33)
    np.testing.assert_allclose(D.layer_norm(x, g, b, eps=0.0), y * g + b, atol=1e-12)
    lp = D.log_softmax(x)
    np.testing.assert_allclose(np.exp(lp).sum(axis=1), 1.0, atol=1e-12)
    np.testing.assert_allclose(lp - lp[:, :1], x - x[:, :1], atol=1e-12)     # shift invariance


def test_update_beam_state_follows_the_trie():
    rng, sids, trie, _ = _tiny(40, B=1)
    V = 64
    level1 = trie.prefixes[1][:, 0]
    prev_tok = level1[:4]
    prev_node = np.array([trie.walk([x]) for x in prev_tok], dtype=np.int32)
    prev_key = Mx.prefix_keys(prev_tok.reshape(-1, 1))
    toks2, _ = trie.lookup(int(prev_node[2]))
    parent = np.array([[2, 2, 0]], dtype=np.int32)
    token = np.array([[int(toks2[0]), 63 if 63 not in toks2 else 62, 5]], dtype=np.int32)
    score = np.array([[-1.0, -2.0, -np.inf]], dtype=np.float32)
    node, key = T.update_beam_state(trie, parent, token, score, prev_node, prev_key, 1, 4)
    assert node[0] == trie.walk([int(prev_tok[2]), int(toks2[0])]) and node[0] >= 0
    assert node[1] == -1 or trie.walk([int(prev_tok[2]), int(token[0, 1])]) == node[1]
    assert node[2] == -1                                  # selected -inf -> dead beam
    assert int(key[0]) == int(Mx.prefix_key([int(prev_tok[2]), int(toks2[0])]))
    assert int(key[2]) == int(Mx.prefix_key([int(prev_tok[0]), 5]))
