"""GPU parity at the benchmark configurations' FULL sizes, in the launch configuration bench.py
times.  The oracle cannot recompute whole outputs there in seconds, so it recomputes sampled outputs
one by one (attention rows, mask rows, whole requests of the top-k) and the rest is covered by
properties that hold at any size."""
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

from gpu_util import DEV, assert_attention_close, assert_log_probs_close, dev, dev_bf16, f64, host_u64  # noqa: E402


@pytest.fixture(scope="module")
def api():
    from paper_2608_00938_b200 import api as _api
    return _api


# ---- configuration 2: cross-attention op sweep ----------------------------------------------------
@pytest.mark.parametrize("B,M,T,H,d", [(64, 256, 512, 8, 64), (64, 1024, 512, 8, 64), (64, 256, 1024, 8, 64),
                                       (64, 1024, 1024, 8, 64),
                                       # head size 128: several items per CTA (both O accumulators and both P column
                                       # sets in turn), one K/V block per item (the paper's shape) and several, ragged T
                                       (16, 1024, 128, 16, 128), (8, 1000, 300, 8, 128), (32, 2048, 1024, 4, 128)])
def test_cross_attn_config2_sampled_rows(api, B, M, T, H, d):
    rng = synth.rng_for(2, M + T + d)
    q = synth.normal_bf16(rng, (B * M, H, d))
    k = synth.normal_bf16(rng, (B, H, T, d))
    v = synth.normal_bf16(rng, (B, H, T, d))
    out = torch.zeros((B * M, H, d), dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros((B * M, H), dtype=torch.float32, device=DEV)
    scale = float(d) ** -0.5
    api.grace_cross_attn(dev_bf16(q), dev_bf16(k), dev_bf16(v), out, scale, lse)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy()
    pick = np.random.default_rng(0)
    rows = pick.integers(0, B * M, size=4096)
    rows[:4] = [0, M - 1, M, B * M - 1]                        # tile and request boundaries
    heads = pick.integers(0, H, size=4096)
    ref = np.stack([OA.cross_attn_row(f64(q[r, h]), f64(k[r // M, h]), f64(v[r // M, h]), scale)
                    for r, h in zip(rows, heads)])
    assert_attention_close(got[rows, heads], ref, f"cross-attn B{B} M{M} T{T}")
    assert np.isfinite(got).all() and np.isfinite(lse.cpu().numpy()).all()
    # a convex combination of the value rows: every output lies inside the per-(request, head) value range
    vmax = torch.from_numpy(synth.bf16_bits_to_f32(v)).amax(dim=2)          # [B, H, d]
    vmin = torch.from_numpy(synth.bf16_bits_to_f32(v)).amin(dim=2)
    g = torch.from_numpy(got).view(B, M, H, d)
    assert (g <= vmax[:, None] + 1e-2).all() and (g >= vmin[:, None] - 1e-2).all()


# ---- configuration 3: self-attention decode op ----------------------------------------------------
@pytest.mark.parametrize("t", [0, 1, 2, 3, 4])
def test_self_attn_config3_sampled_rows(api, t):
    B, M, H, d, L = 32, 2048, 8, 64, 5
    R = B * M
    rng = synth.rng_for(3, t)
    sizes = [M] * (t + 1)
    kc = np.zeros((L, R, H, d), dtype=np.uint16)
    vc = np.zeros((L, R, H, d), dtype=np.uint16)
    parents = np.zeros((L, R), dtype=np.int32)
    for j in range(t):
        kc[j] = synth.normal_bf16(rng, (R, H, d))
        vc[j] = synth.normal_bf16(rng, (R, H, d))
    for j in range(1, t + 1):
        parents[j] = synth.uniform_parents(rng, B, M, M)
    qkv = synth.normal_bf16(rng, (R, 3, H, d))
    d_kc, d_vc = dev_bf16(kc), dev_bf16(vc)
    out = torch.zeros((R, H, d), dtype=torch.bfloat16, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    api.grace_self_attn(dev_bf16(qkv), d_kc, d_vc, dev(parents), sizes, out, B, t, 0.125, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    got = out.float().cpu().numpy()
    rows = np.random.default_rng(1).integers(0, R, size=1024)
    rows[:3] = [0, M - 1, R - 1]
    kc64, vc64 = synth.bf16_bits_to_f32(kc), synth.bf16_bits_to_f32(vc)
    par_list = [None] + [parents[j] for j in range(1, t + 1)]
    ref = np.stack([OA.self_attn_row(f64(qkv[r]), kc64, vc64, par_list, sizes, t, r // M, r % M, 0.125) for r in rows])
    assert_attention_close(got[rows], ref, f"self-attn T_self={t + 1}")
    # cache write: slab t is exactly k, v of the rows (bit-exact), older slabs untouched
    assert torch.equal(d_kc[t].view(torch.int16).cpu(), torch.from_numpy(qkv[:, 1].view(np.int16)))
    assert torch.equal(d_vc[t].view(torch.int16).cpu(), torch.from_numpy(qkv[:, 2].view(np.int16)))
    if t:
        assert torch.equal(d_kc[:t].view(torch.int16).cpu(), torch.from_numpy(kc[:t].view(np.int16)))


# ---- configuration 4: GTM mask + beam top-k ---------------------------------------------------------
@pytest.fixture(scope="module")
def config4():
    V, L, n = 1024, 4, 1_000_000
    rng = synth.rng_for(4, 0)
    sids = synth.catalog(rng, n, V, L)
    return dict(V=V, L=L, sids=sids, trie=SidTrie(sids, V), rng=rng)


@pytest.mark.parametrize("depth,M", [(1, 1024), (2, 2048), (3, 2048)])
def test_mask_then_topk_config4(api, config4, depth, M):
    V, L, sids, trie = config4["V"], config4["L"], config4["sids"], config4["trie"]
    B, K = 32, 2048
    rng = synth.rng_for(4, 10 + depth)
    bits, base, level_start = api.grace_trie_build_dense(sids, V)
    trie_s = api.make_trie(dev(bits), dev(base), V, L, trie.num_nodes)
    elig, blooms, node, key, score = [], [], np.full((B, M), -1, np.int32), np.zeros((B, M), np.uint64), []
    for b in range(B):
        e = synth.eligible_subset(rng, sids.shape[0], 0.2)
        elig.append(e)
        blooms.append(api.grace_bloom_build(sids, V, e, 22, 4))
        pref = synth.beam_prefixes_from_sids(rng, sids[e], depth, M)
        n = pref.shape[0]
        level = trie.prefixes[depth]
        rank = OM._rows_rank(level, pref.astype(np.int64))                  # node id = level start + lexicographic rank
        node[b, :n] = trie.level_start[depth] + rank
        key[b, :n] = OM.prefix_keys(pref)
        score.append(synth.descending_scores(rng, M, depth))
    score = np.concatenate(score)
    matcher = api.make_matcher(api.MATCH_PREFIX_BLOOM, dev(np.stack(blooms)), 22, 4)
    logp = synth.logp_rows(rng, B * M, V)
    d_logp = dev(logp)
    cand = torch.empty((B * M, V), device=DEV)
    allow = torch.zeros((B * M, V // 64), dtype=torch.int64, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    api.grace_gtm_mask(d_logp, dev(score), dev(node.reshape(-1)), dev(key.reshape(-1)), trie_s, matcher, cand, allow,
                       B, M, depth, status)
    ws = torch.empty(api.grace_beam_topk_workspace_bytes(B, M * V, K), dtype=torch.uint8, device=DEV)
    o_score = torch.empty((B, K), device=DEV)
    o_flat = torch.empty((B, K), dtype=torch.int32, device=DEV)
    o_par, o_tok = torch.empty_like(o_flat), torch.empty_like(o_flat)
    api.grace_beam_topk(cand.view(B, M * V), K, V, o_score, o_flat, o_par, o_tok, ws, status)
    torch.cuda.synchronize()
    assert status.item() & (api.DEV_NAN | api.DEV_BAD_INDEX) == 0
    h_cand = cand.cpu().numpy()
    h_allow = host_u64(allow)
    # mask: sampled rows recomputed by the oracle (whole rows, bit-exact), oracle's own Bloom filter
    o_blooms = {}
    rows = np.random.default_rng(2).integers(0, B * M, size=192)
    rows[:2] = [0, B * M - 1]
    for r in rows:
        b = r // M
        if b not in o_blooms:
            o_blooms[b] = OM.build_prefix_bloom(sids, elig[b], 22, 4)
            assert np.array_equal(o_blooms[b].words, blooms[b])
        c_ref, a_ref, _ = OG.gtm_mask(logp[r:r + 1], score[r:r + 1], node.reshape(-1)[r:r + 1],
                                      key.reshape(-1)[r:r + 1], depth, trie, _OneRequest(o_blooms[b]), 1, 1)
        assert np.array_equal(h_cand[r].view(np.uint32), c_ref[0].view(np.uint32))
        assert np.array_equal(h_allow[r], OG.pack_allow_bits(a_ref)[0])
    # properties at full size: finite <=> allowed, dead rows fully masked, allowed implies catalog child
    finite = np.isfinite(h_cand)
    unpacked = np.unpackbits(h_allow.view(np.uint8), axis=1, bitorder="little").astype(bool)
    assert np.array_equal(finite, unpacked)
    assert not finite[node.reshape(-1) < 0].any()
    child_bits = np.unpackbits(bits[np.maximum(node.reshape(-1), 0)].view(np.uint8), axis=1, bitorder="little").astype(bool)
    assert not (finite & ~child_bits).any()
    # top-k: three whole requests against the oracle (exact), all requests against order properties
    for b in (0, 13, B - 1):
        s_ref, f_ref, p_ref, t_ref = OT.beam_topk(h_cand.reshape(B, M * V)[b:b + 1], K, V)
        assert np.array_equal(o_flat[b].cpu().numpy(), f_ref[0])
        assert np.array_equal(o_score[b].cpu().numpy().view(np.uint32), s_ref[0].view(np.uint32))
        assert np.array_equal(o_par[b].cpu().numpy(), p_ref[0]) and np.array_equal(o_tok[b].cpu().numpy(), t_ref[0])
    sc = o_score.cpu().numpy()
    fl = o_flat.cpu().numpy().astype(np.int64)
    assert (sc[:, 1:] <= sc[:, :-1]).all()
    assert all(len(set(fl[b])) == K for b in range(B))
    flat_cand = h_cand.reshape(B, M * V)
    assert np.array_equal(np.take_along_axis(flat_cand, fl, axis=1).view(np.uint32), sc.view(np.uint32))
    n_finite = finite.reshape(B, -1).sum(axis=1)
    assert np.array_equal(np.isfinite(sc).sum(axis=1), np.minimum(n_finite, K))       # all finite taken before any -inf
    kth = sc[:, -1]
    for b in range(B):
        rest = np.delete(flat_cand[b], fl[b])
        assert rest.size == 0 or rest.max() <= kth[b]


class _OneRequest(OG.PrefixBloomMatcher):
    """Oracle matcher holding the one Bloom filter of the request a sampled row belongs to."""

    def __init__(self, bloom):
        super().__init__([bloom])


def test_topk_config4_dense_unmasked(api):
    """Variant (i): top-k alone on dense, all-finite candidates (the worst case for selection)."""
    B, M, V, K = 32, 2048, 1024, 2048
    rng = synth.rng_for(4, 20)
    cand = np.empty((B, M * V), dtype=np.float32)
    for b in range(B):
        cand[b] = (synth.descending_scores(rng, M, 2)[:, None] + synth.logp_rows(rng, M, V)).reshape(-1)
    d_cand = dev(cand)
    ws = torch.empty(api.grace_beam_topk_workspace_bytes(B, M * V, K), dtype=torch.uint8, device=DEV)
    o_score = torch.empty((B, K), device=DEV)
    o_flat = torch.empty((B, K), dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    api.grace_beam_topk(d_cand, K, V, o_score, o_flat, None, None, ws, status)
    torch.cuda.synchronize()
    assert status.item() & (api.DEV_NAN | api.DEV_BAD_INDEX) == 0
    for b in (0, 7, 31):
        s_ref, f_ref, _, _ = OT.beam_topk(cand[b:b + 1], K, V)
        assert np.array_equal(o_flat[b].cpu().numpy(), f_ref[0])
        assert np.array_equal(o_score[b].cpu().numpy().view(np.uint32), s_ref[0].view(np.uint32))
    sc, fl = o_score.cpu().numpy(), o_flat.cpu().numpy().astype(np.int64)
    assert (sc[:, 1:] <= sc[:, :-1]).all()
    for b in range(B):
        assert (cand[b] > sc[b, -1]).sum() < K <= (cand[b] >= sc[b, -1]).sum()


# ---- configuration 5: the full decoder step at serving scale ----------------------------------------
@pytest.mark.parametrize("workload,schedule,modes", [
    ("cfg5", None, (False, True)),                        # fp32 and bf16 residual stream, same tolerance
    ("paper", None, (True,)),                             # the paper's decoder shape, dynamic beams (1,512,1024,1024)
    ("paper", (1, 1024, 1024, 1024), (True,)),            # its fixed schedule: step 0 wider than the codebook
])
def test_decode_step_full_size_teacher_forced_on_one_request(workload, schedule, modes):
    """The bench workloads at full size (cfg5: 32 requests x beam 2048, 4 layers, V = 2048; paper: 16 requests,
    3 layers, 16 heads of 128, V = 512; 1M-SID catalog, Bloom matcher): the library decodes the whole batch; the
    oracle decodes request 0 alone (requests never interact) and the library's request-0 rows are checked step
    by step, each step starting from the oracle's beam state."""
    import bench
    from oracle import decoder as OD
    from paper_2608_00938_b200 import api
    from paper_2608_00938_b200.decoder import Decoder
    cfg = dict(bench.WORKLOADS[workload])
    if schedule is not None:
        cfg["schedule"], cfg["final_k"] = schedule, schedule[-1]
    inp = bench.make_inputs(cfg, 0)
    sids, V, L, B = inp["sids"], cfg["V"], cfg["L"], cfg["B"]
    sizes = list(cfg["schedule"]) + [cfg["final_k"]]
    trie = SidTrie(sids, V)
    bloom0 = OM.build_prefix_bloom(sids, inp["elig"][0], cfg["bloom_log2"], cfg["bloom_hashes"])
    record = []
    OD.beam_search(inp["weights"], inp["shp"], synth.bf16_bits_to_f32(inp["enc_bits"][:1]), trie,
                   OG.PrefixBloomMatcher([bloom0]), cfg["schedule"], cfg["final_k"], record=record)

    bits, base, level_start = api.grace_trie_build_dense(sids, V)
    assert int(level_start[-1]) == trie.num_nodes
    blooms = np.stack([api.grace_bloom_build(sids, V, e, cfg["bloom_log2"], cfg["bloom_hashes"]) for e in inp["elig"]])
    assert np.array_equal(blooms[0], bloom0.words)
    for residual_bf16 in modes:
        dec = Decoder(n_layers=cfg["n_layers"], d_model=cfg["d_model"], n_heads=cfg["H"], d_head=cfg["d_h"],
                      d_ffn=cfg["d_ffn"], V=V, L=L, T_ctx=cfg["T_ctx"], B=B, beam_sizes=sizes, weights=inp["weights"],
                      trie_bits=bits, trie_base=base, num_nodes=trie.num_nodes,
                      matcher=(api.MATCH_PREFIX_BLOOM, blooms, cfg["bloom_log2"], cfg["bloom_hashes"]), device=DEV,
                      separate_cand=True, residual_bf16=residual_bf16)
        dec.project_cross_kv(dev_bf16(inp["enc_bits"]))
        dec.reset()
        for t in range(L):
            step = record[t]
            M, K = sizes[t], sizes[t + 1]
            cur, nxt = t & 1, (t + 1) & 1
            # request 0 occupies rows 0..M-1 (request-major); the other 31 requests run free
            dec.token[cur][:M].copy_(dev(step["tokens"].astype(np.int32)))
            dec.score[cur][:M].copy_(dev(step["score"]))
            dec.node[cur][:M].copy_(dev(step["node"]))
            dec.key[cur][:M].copy_(dev(step["key"]))
            if t > 0:
                dec.parents[t, :M].copy_(dev(record[t - 1]["out_parent"].reshape(-1)))
            dec.step(t)
            torch.cuda.synchronize()
            assert dec.d_status.item() & ~api.DEV_TOPK_EXACT_PATH == 0
            logp = dec.log_probs(M).cpu().numpy()
            live = step["node"] >= 0                 # dead beams are never normalised (everything is masked)
            assert_log_probs_close(logp[live], step["logp"][live], f"step {t}")
            cand = dec.cand[:M].cpu().numpy()
            assert np.array_equal(np.isfinite(cand), step["allow"])                       # same mask as the oracle
            assert np.array_equal(cand[step["allow"]], (step["score"][:, None] + logp)[step["allow"]])
            sc, flat, par, tok = OT.beam_topk(cand.reshape(1, M * V), K, V)               # exact on the GPU's own candidates
            assert np.array_equal(dec.out_flat[:K].cpu().numpy(), flat[0])
            assert np.array_equal(dec.score[nxt][:K].cpu().numpy().view(np.uint32), sc[0].view(np.uint32))
            assert np.array_equal(dec.parents[t + 1, :K].cpu().numpy(), par[0])
            assert np.array_equal(dec.token[nxt][:K].cpu().numpy(), tok[0])
            node_ref, key_ref = OT.update_beam_state(trie, par, tok, sc, step["node"], step["key"], t, M)
            assert np.array_equal(dec.node[nxt][:K].cpu().numpy(), node_ref)
            assert np.array_equal(dec.key[nxt][:K].cpu().numpy().view(np.uint64), key_ref)
            # every request (free-running ones too): selected scores sorted, live beams sit on catalog nodes
            all_sc = dec.score[nxt][:B * K].view(B, K).cpu().numpy()
            assert (all_sc[:, 1:] <= all_sc[:, :-1]).all()
            all_node = dec.node[nxt][:B * K].cpu().numpy()
            assert np.array_equal(all_node >= 0, np.isfinite(all_sc.reshape(-1)))
            assert ((all_node < 0) | ((all_node >= trie.level_start[t + 1]) & (all_node < trie.level_start[t + 2]))).all()
        # the emitted SIDs of every request are catalog SIDs whose prefixes all pass that request's Bloom filter
        g_sids, g_score, g_node = dec.results()
        catalog_keys = set(OM.prefix_keys(sids).tolist())
        for b in (0, 5, B - 1):
            valid = np.isfinite(g_score[b])
            assert valid.sum() > 0
            keys = OM.prefix_keys(g_sids[b][valid])
            assert all(int(x) in catalog_keys for x in keys)
            bl = OM.PrefixBloom(cfg["bloom_log2"], cfg["bloom_hashes"])
            bl.words = blooms[b]
            for l in range(1, L + 1):
                assert bl.contains(OM.prefix_keys(g_sids[b][valid][:, :l])).all()
        del dec
        torch.cuda.empty_cache()


@pytest.mark.parametrize("workload", ["cfg5", "paper"])
def test_bench_decode_path_equals_the_materialised_path_at_config5(workload):
    """The decoder exactly as bench.py builds it (bf16 residual stream; the constraint ahead of a logits GEMM that
    stores the allowed logits only, every step selected through the allow bits) against the same decoder with the
    whole logits tensor written, and with every step materialised: free-running over all requests, at serving
    scale and at the paper's decoder shape (head size 128, V = 512), the final beams must agree bit for bit."""
    import bench
    cfg = dict(bench.WORKLOADS[workload])
    inp = bench.make_inputs(cfg, 0)
    enc = dev_bf16(inp["enc_bits"])
    B, K = cfg["B"], cfg["final_k"]
    outs = []
    # bench's own form (the constraint before a logits GEMM that stores allowed logits only, on every step); the
    # whole logits tensor written, candidates materialised on the dense trie level and read through allow bits on
    # the sparse ones; everything materialised
    for how in (dict(), dict(logits_allowed_only=False), dict(materialize_cand=True)):
        dec = bench.build_decoder(cfg, inp, DEV, residual_bf16=True, **how)
        if not how:
            assert dec.allow_bits is not None and dec.logits_allowed_only and dec.masked_from_step == 0
        elif "logits_allowed_only" in how:
            assert dec.allow_bits is not None and 0 < dec.masked_from_step < cfg["L"]      # a mixed schedule
        dec.project_cross_kv(enc)
        dec.reset(); dec.decode()
        torch.cuda.synchronize()
        fin = dec.L & 1
        assert dec.d_status.item() & ~8 == 0                                              # 8: informational
        outs.append((dec.score[fin][:B * K].clone(), dec.key[fin][:B * K].clone(), dec.node[fin][:B * K].clone()))
        del dec
        torch.cuda.empty_cache()
    assert torch.isfinite(outs[0][0]).sum() > B * K // 2
    for other in outs[1:]:
        assert torch.equal(outs[0][0].view(torch.int32), other[0].view(torch.int32))
        assert torch.equal(outs[0][1], other[1]) and torch.equal(outs[0][2], other[2])
    if workload != "cfg5":
        return
    # the same pair with the LayerNorms as kernels of their own (the logits GEMM then reads the normalised copy)
    outs = []
    for how in (dict(), dict(logits_allowed_only=False)):
        dec = bench.build_decoder(cfg, inp, DEV, residual_bf16=True, fold_layer_norm=False, **how)
        dec.project_cross_kv(enc)
        dec.reset(); dec.decode()
        torch.cuda.synchronize()
        fin = dec.L & 1
        assert dec.d_status.item() & ~8 == 0
        outs.append((dec.score[fin][:B * K].clone(), dec.key[fin][:B * K].clone(), dec.node[fin][:B * K].clone()))
        del dec
        torch.cuda.empty_cache()
    assert torch.isfinite(outs[0][0]).sum() > B * K // 2
    assert torch.equal(outs[0][0].view(torch.int32), outs[1][0].view(torch.int32))
    assert torch.equal(outs[0][1], outs[1][1]) and torch.equal(outs[0][2], outs[1][2])


def test_bench_decoder_teacher_forced_against_the_oracle_at_config5():
    """The decoder exactly as bench.py builds it (bf16 residual stream, LayerNorm folded into the GEMMs over a
    centred stream, cache held in place, the constraint ahead of a logits GEMM that stores the allowed logits
    only), and its form with the whole logits tensor written and candidates materialised on the dense trie
    level, teacher-forced on request 0 against the oracle's decode of that request:
    at every step the allow bits / finite candidates equal the oracle's mask, the log-probabilities agree
    within the decoder tolerance, and the selection, parents, tokens, nodes and keys equal the oracle's
    top-k and state update run on the GPU's own candidates, bit for bit."""
    import bench
    from oracle import decoder as OD
    from paper_2608_00938_b200 import api
    cfg = dict(bench.CFG5)
    inp = bench.make_inputs(cfg, 0)
    sids, V, L, B = inp["sids"], cfg["V"], cfg["L"], cfg["B"]
    sizes = list(cfg["schedule"]) + [cfg["final_k"]]
    trie = SidTrie(sids, V)
    bloom0 = OM.build_prefix_bloom(sids, inp["elig"][0], cfg["bloom_log2"], cfg["bloom_hashes"])
    record = []
    OD.beam_search(inp["weights"], inp["shp"], synth.bf16_bits_to_f32(inp["enc_bits"][:1]), trie,
                   OG.PrefixBloomMatcher([bloom0]), cfg["schedule"], cfg["final_k"], record=record)
    # bench's own form (constraint first, allowed logits only, every step through the allow bits) and the form that
    # writes the whole logits tensor (dense trie level materialised, sparse levels through the allow bits)
    for how in (dict(), dict(logits_allowed_only=False)):
        dec = bench.build_decoder(cfg, inp, DEV, residual_bf16=True, **how)
        if not how:
            assert dec.allow_bits is not None and dec.logits_allowed_only and dec.masked_from_step == 0
        else:
            assert dec.allow_bits is not None and 0 < dec.masked_from_step < L   # both candidate paths are exercised
        _teacher_force_bench_decoder(dec, record, trie, inp, sizes, V, L, api)
        del dec
        torch.cuda.empty_cache()


def _teacher_force_bench_decoder(dec, record, trie, inp, sizes, V, L, api):
    dec.project_cross_kv(dev_bf16(inp["enc_bits"]))
    dec.reset()
    for t in range(L):
        step = record[t]
        M, K = sizes[t], sizes[t + 1]
        cur, nxt = t & 1, (t + 1) & 1
        dec.token[cur][:M].copy_(dev(step["tokens"].astype(np.int32)))
        dec.score[cur][:M].copy_(dev(step["score"]))
        dec.node[cur][:M].copy_(dev(step["node"]))
        dec.key[cur][:M].copy_(dev(step["key"]))
        if t > 0:
            dec.parents[t, :M].copy_(dev(record[t - 1]["out_parent"].reshape(-1)))
        dec.step(t)
        torch.cuda.synchronize()
        assert dec.d_status.item() & ~api.DEV_TOPK_EXACT_PATH == 0
        live = step["node"] >= 0
        score = step["score"].astype(np.float32)
        if t < dec.masked_from_step:
            cand = dec.cand[:M].cpu().numpy()                                    # written in place of the logits
            assert np.array_equal(np.isfinite(cand), step["allow"])
            got_logp = (cand - score[:, None])[step["allow"]]
            ref_logp = step["logp"][step["allow"]]
        else:
            bits = dec.allow_bits[:M].cpu().numpy().view(np.uint64)
            assert np.array_equal(bits, OG.pack_allow_bits(step["allow"]))
            logits = dec.logp[:M].cpu().numpy()
            lse = dec.row_lse[:M].cpu().numpy()
            logp = logits - lse[:, None]
            cand = np.where(step["allow"], score[:, None] + logp, np.float32(-np.inf)).astype(np.float32)
            if dec.logits_allowed_only:          # the GEMM stored the allowed logits only: the rest of logp is stale
                got_logp, ref_logp = logp[step["allow"]], step["logp"][step["allow"]]
            else:
                got_logp, ref_logp = logp[live], step["logp"][live]
        assert_log_probs_close(got_logp, ref_logp, f"bench decoder step {t}")
        sc, flat, par, tok = OT.beam_topk(cand.reshape(1, M * V), K, V)           # exact, on the GPU's own candidates
        assert np.array_equal(dec.out_flat[:K].cpu().numpy(), flat[0])
        assert np.array_equal(dec.score[nxt][:K].cpu().numpy().view(np.uint32), sc[0].view(np.uint32))
        assert np.array_equal(dec.parents[t + 1, :K].cpu().numpy(), par[0])
        assert np.array_equal(dec.token[nxt][:K].cpu().numpy(), tok[0])
        node_ref, key_ref = OT.update_beam_state(trie, par, tok, sc, step["node"], step["key"], t, M)
        assert np.array_equal(dec.node[nxt][:K].cpu().numpy(), node_ref)
        assert np.array_equal(dec.key[nxt][:K].cpu().numpy().view(np.uint64), key_ref)
