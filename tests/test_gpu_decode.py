"""GPU parity of grace_decode_step against the oracle's constrained beam search
(configuration 1: one request, beam 16, 2-layer decoder, 2,000-SID catalog,
node-bitmask matcher), teacher-forced step by step, plus a free-running decode."""
import numpy as np
import pytest
import torch

import synth
from oracle import decoder as OD
from oracle import gtm as OG
from oracle import matchers as OM
from oracle import topk as OT
from oracle.sid_trie import SidTrie

pytestmark = pytest.mark.gpu

from gpu_util import DEV, assert_log_probs_close, dev  # noqa: E402


def _config1(B=1, matcher_kind="node", schedule=(1, 16, 16), final_k=16, n_sids=2000, V=64, seed_variant=0,
             std=0.02, shape=(2, 128, 4, 32, 512, 128), T_ctx=64, ln_affine=False, embed_offset=0.0):
    """shape = (layers, d_model, heads, head size, FFN width, encoder width).  ln_affine: LayerNorm gains and
    biases away from (1, 0), so that a folded LayerNorm has something to fold.  embed_offset: a constant added to
    every embedding row (a per-row shift of the residual stream, which no LayerNorm sees)."""
    rng = synth.rng_for(1, seed_variant)
    L = len(schedule)
    sids = synth.catalog(rng, n_sids, V, L)
    trie = SidTrie(sids, V)
    elig = [synth.eligible_subset(rng, n_sids, 0.3) for _ in range(B)]
    shp = synth.DecoderShape(*shape, V, L)
    w = synth.decoder_weights(rng, shp, std=std, as_bf16=True)
    if ln_affine:
        d = shape[1]
        for holder, names in [(w, ("lnf",))] + [(lw, ("ln1", "ln2", "ln3")) for lw in w["layers"]]:
            for n in names:
                holder[n + "_g"] = (1.0 + 0.25 * synth.normal_f32(rng, d)).astype(np.float32)
                holder[n + "_b"] = (0.3 * synth.normal_f32(rng, d)).astype(np.float32)
    if embed_offset:
        w["embed"] = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(
            (np.asarray(w["embed"], np.float32) + np.float32(embed_offset)).astype(np.float32)))
    enc = synth.bf16_bits_to_f32(synth.normal_bf16(rng, (B, T_ctx, shape[5])))
    return dict(sids=sids, trie=trie, elig=elig, shp=shp, w=w, enc=enc, schedule=schedule, final_k=final_k, B=B,
                matcher_kind=matcher_kind)


def _make_gpu_decoder(cfg, separate_cand=True, residual_bf16=False):
    # residual_bf16: False, True (the default bf16 path: LayerNorms folded into the GEMMs over a centred stream),
    # "uncentred" (folded, column sums carry the row means) or "kernel" (LayerNorm kernels of their own)
    fold = {"uncentred": dict(fold_layer_norm=True, centre_stream=False),
            "kernel": dict(fold_layer_norm=False)}.get(residual_bf16, {})
    residual_bf16 = bool(residual_bf16)
    from paper_2608_00938_b200 import api
    from paper_2608_00938_b200.decoder import Decoder
    shp, sids, trie = cfg["shp"], cfg["sids"], cfg["trie"]
    bits, base, level_start = api.grace_trie_build_dense(sids, shp.V)
    if cfg["matcher_kind"] == "node":
        mb = np.stack([api.grace_node_bitmask_build(sids, shp.V, e, trie.num_nodes) for e in cfg["elig"]])
        matcher = (api.MATCH_NODE_BITMASK, mb, 0, 0)
    else:
        mb = np.stack([api.grace_bloom_build(sids, shp.V, e, 14, 4) for e in cfg["elig"]])
        matcher = (api.MATCH_PREFIX_BLOOM, mb, 14, 4)
    dec = Decoder(n_layers=shp.n_layers, d_model=shp.d_model, n_heads=shp.n_heads, d_head=shp.d_head,
                  d_ffn=shp.d_ffn, V=shp.V, L=shp.L, T_ctx=cfg["enc"].shape[1], B=cfg["B"],
                  beam_sizes=list(cfg["schedule"]) + [cfg["final_k"]], weights=cfg["w"], trie_bits=bits,
                  trie_base=base, num_nodes=trie.num_nodes, matcher=matcher, device=DEV, separate_cand=separate_cand,
                  residual_bf16=residual_bf16, **fold)
    dec.project_cross_kv(torch.from_numpy(cfg["enc"]).to(DEV).to(torch.bfloat16))
    return dec, api


def _oracle_matcher(cfg):
    sids, trie = cfg["sids"], cfg["trie"]
    if cfg["matcher_kind"] == "node":
        return OG.NodeBitmaskMatcher(np.stack([OM.node_eligibility(trie, sids, e) for e in cfg["elig"]]))
    return OG.PrefixBloomMatcher([OM.build_prefix_bloom(sids, e, 14, 4) for e in cfg["elig"]])


# the paper's decoder geometry, narrowed: 16 heads of 128 (rows of 2048), 128 context tokens, 4 levels
_PAPER_LIKE = dict(shape=(2, 256, 16, 128, 512, 256), T_ctx=128, n_sids=4000)


@pytest.mark.parametrize("B,kind,schedule,final_k,residual_bf16,extra", [
    (1, "node", (1, 16, 16), 16, False, {}),     # configuration 1
    (3, "bloom", (1, 40, 24), 32, False, {}),    # several requests, dynamic per-step beam sizes, Bloom matcher
    (3, "bloom", (1, 40, 24), 32, True, {}),     # the same with the residual stream held in bf16
    (3, "bloom", (1, 40, 24), 32, "uncentred", {}),
    (3, "bloom", (1, 40, 24), 32, "kernel", {}),
    (3, "bloom", (1, 40, 24), 32, True, dict(ln_affine=True)),          # gains and biases that the fold must carry
    (3, "bloom", (1, 40, 24), 32, "uncentred", dict(ln_affine=True)),
    (3, "bloom", (1, 40, 24), 32, "kernel", dict(ln_affine=True)),
    (3, "bloom", (1, 40, 24), 32, False, dict(ln_affine=True)),          # fp32 stream
    # a stream whose rows sit at a mean of 0.5 with a spread of a few hundredths: a bf16 stream that holds the mean
    # loses most of the signal (measured: rms error 0.04 x the logit spread for the uncentred bf16 variants); the
    # centred stream never sees the mean (0.006 x), the fp32 stream can hold it (0.004 x)
    (3, "bloom", (1, 40, 24), 32, True, dict(ln_affine=True, embed_offset=0.5)),
    (3, "bloom", (1, 40, 24), 32, False, dict(ln_affine=True, embed_offset=0.5)),
    (2, "bloom", (1, 24, 48, 48), 48, True, _PAPER_LIKE),   # dynamic schedule over 4 levels, head size 128
    (2, "node", (1, 100, 80), 80, True, {}),      # step 0 asks for more beams than there are tokens (fixed-schedule shape)
])
def test_decode_step_teacher_forced(B, kind, schedule, final_k, residual_bf16, extra):
    cfg = _config1(B=B, matcher_kind=kind, schedule=schedule, final_k=final_k, **extra)
    shp, trie = cfg["shp"], cfg["trie"]
    record = []
    OD.beam_search(cfg["w"], shp, cfg["enc"], trie, _oracle_matcher(cfg), schedule, final_k, record=record)
    dec, api = _make_gpu_decoder(cfg, residual_bf16=residual_bf16)
    dec.reset()
    V, L = shp.V, shp.L
    sizes = list(schedule) + [final_k]
    for t in range(L):
        step = record[t]
        M, K = sizes[t], sizes[t + 1]
        R = B * M
        cur, nxt = t & 1, (t + 1) & 1
        # teacher forcing: the step starts from the oracle's beam state (caches come from the GPU's own
        # earlier steps, which ran on the same tokens and parents)
        dec.token[cur][:R].copy_(dev(step["tokens"].astype(np.int32)))
        dec.score[cur][:R].copy_(dev(step["score"]))
        dec.node[cur][:R].copy_(dev(step["node"]))
        dec.key[cur][:R].copy_(dev(step["key"]))
        if t > 0:
            dec.parents[t, :R].copy_(dev(record[t - 1]["out_parent"].reshape(-1)))
        dec.step(t)
        torch.cuda.synchronize()
        assert dec.d_status.item() & ~api.DEV_TOPK_EXACT_PATH == 0
        # log-probabilities: bf16 pipeline vs the fp64 oracle on the same bf16-valued weights
        logp = dec.log_probs(R).cpu().numpy()
        live = step["node"] >= 0                 # dead beams are never normalised (everything is masked)
        assert_log_probs_close(logp[live], step["logp"][live], f"step {t}")
        np.testing.assert_allclose(np.exp(logp[live].astype(np.float64)).sum(1), 1.0, atol=1e-4)
        # the mask is an integer decision on exact inputs: identical to the oracle's
        cand = dec.cand[:R].cpu().numpy()
        assert np.array_equal(np.isfinite(cand), step["allow"])
        assert np.array_equal(cand[step["allow"]], (step["score"][:, None] + logp)[step["allow"]])
        # selection and state update: exact against the oracle run on the GPU's own candidates
        sc, flat, par, tok = OT.beam_topk(cand.reshape(B, M * V), K, V)
        assert np.array_equal(dec.out_flat[:B * K].cpu().numpy().reshape(B, K), flat)
        assert np.array_equal(dec.score[nxt][:B * K].cpu().numpy().view(np.uint32).reshape(B, K), sc.view(np.uint32))
        assert np.array_equal(dec.parents[t + 1, :B * K].cpu().numpy().reshape(B, K), par)
        assert np.array_equal(dec.token[nxt][:B * K].cpu().numpy().reshape(B, K), tok)
        node_ref, key_ref = OT.update_beam_state(trie, par, tok, sc, step["node"], step["key"], t, M)
        assert np.array_equal(dec.node[nxt][:B * K].cpu().numpy(), node_ref)
        assert np.array_equal(dec.key[nxt][:B * K].cpu().numpy().view(np.uint64), key_ref)


def test_free_running_decode_emits_only_eligible_catalog_sids():
    """Wide beams on a small catalog: the search is exhaustive, so GPU and oracle must return the same
    set of SIDs; every emitted SID is in the catalog and passes the matcher at every prefix."""
    cfg = _config1(B=2, matcher_kind="node", schedule=(1, 64, 64), final_k=64, n_sids=60, std=0.3)
    shp, trie, sids = cfg["shp"], cfg["trie"], cfg["sids"]
    out = OD.beam_search(cfg["w"], shp, cfg["enc"], trie, _oracle_matcher(cfg), cfg["schedule"], cfg["final_k"])
    dec, api = _make_gpu_decoder(cfg, separate_cand=False)
    dec.reset()
    dec.decode()
    torch.cuda.synchronize()
    assert dec.d_status.item() & ~api.DEV_TOPK_EXACT_PATH == 0
    g_sids, g_score, g_node = dec.results()
    for b in range(cfg["B"]):
        good = {tuple(s) for s, e in zip(sids.tolist(), cfg["elig"][b]) if e}
        valid = np.isfinite(g_score[b])
        got = [tuple(s) for s in g_sids[b][valid].tolist()]
        want = [tuple(s) for s in out["sids"][b][out["valid"][b]].tolist()]
        assert set(got) == set(want) == good
        assert all(trie.walk(s) == n for s, n in zip(got, g_node[b][valid]))
        assert (g_score[b][1:] <= g_score[b][:-1]).all()
        # weights of std 0.3 give scores down to -35: bf16 activations carry ~1% of that
        np.testing.assert_allclose(np.sort(g_score[b][valid]), np.sort(out["score"][b][out["valid"][b]]), atol=3e-2, rtol=5e-2)


def test_whole_decode_loop_replays_from_a_cuda_graph():
    """The decode loop enqueues kernels only (no allocation, no host synchronisation, tensor maps passed by
    value), so all steps can be captured once into a CUDA graph and replayed (Section 5: the full fixed-length
    decoding loop is captured as one graph).  The replay must reproduce the eager results bit for bit."""
    cfg = _config1(B=3, matcher_kind="bloom", schedule=(1, 40, 24), final_k=32)
    dec, api = _make_gpu_decoder(cfg, separate_cand=False)
    dec.reset(); dec.decode()                                   # eager run (also warms every lazy attribute set-up)
    torch.cuda.synchronize()
    fin = dec.L & 1
    n = cfg["B"] * cfg["final_k"]
    eager = (dec.score[fin][:n].clone(), dec.key[fin][:n].clone(), dec.node[fin][:n].clone())
    launches0 = api.grace_kernel_launch_count()
    graph = torch.cuda.CUDAGraph()
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            dec.reset(); dec.decode()
    per_loop = api.grace_kernel_launch_count() - launches0
    assert per_loop > 0
    for buf in (dec.score[fin], dec.key[fin], dec.node[fin]):
        buf.zero_()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert api.grace_kernel_launch_count() - launches0 == per_loop          # replays launch nothing from the host
    assert torch.equal(dec.score[fin][:n].view(torch.int32), eager[0].view(torch.int32))
    assert torch.equal(dec.key[fin][:n], eager[1]) and torch.equal(dec.node[fin][:n], eager[2])
    assert dec.d_status.item() & ~api.DEV_TOPK_EXACT_PATH == 0


def test_serving_loop_with_overlapped_host_copies_matches_one_batch_at_a_time():
    """Decoder.serve: inputs arrive from pinned host memory on a copy stream (batch i+1 under batch i's compute),
    results leave on it.  Every batch must come out exactly as when it is decoded alone."""
    cfg = _config1(B=3, matcher_kind="bloom", schedule=(1, 40, 24), final_k=32)
    dec, api = _make_gpu_decoder(cfg, separate_cand=False, residual_bf16=True)
    rng = synth.rng_for(1, 77)
    n_batches, n = 5, cfg["B"] * cfg["final_k"]
    fin = dec.L & 1
    encs = [synth.normal_bf16(rng, cfg["enc"].shape) for _ in range(n_batches)]
    alone = []
    for e in encs:
        dec.project_cross_kv(torch.from_numpy(e.view(np.int16)).to(DEV).view(torch.bfloat16))
        dec.reset(); dec.decode()
        torch.cuda.synchronize()
        alone.append((dec.score[fin][:n].cpu(), dec.key[fin][:n].cpu(), dec.node[fin][:n].cpu()))
    assert not torch.equal(alone[0][1], alone[1][1])                       # the batches really differ
    hosts = [torch.from_numpy(e.view(np.int16).copy()).view(torch.bfloat16).pin_memory() for e in encs]
    outs = [dict(score=torch.empty(n, dtype=torch.float32).pin_memory(), key=torch.empty(n, dtype=torch.int64).pin_memory(),
                 node=torch.empty(n, dtype=torch.int32).pin_memory()) for _ in range(n_batches)]
    dec.serve(hosts, outs)
    for i in range(n_batches):
        assert torch.equal(outs[i]["score"].view(torch.int32), alone[i][0].view(torch.int32)), i
        assert torch.equal(outs[i]["key"], alone[i][1]) and torch.equal(outs[i]["node"], alone[i][2]), i
    assert dec.d_status.item() & ~api.DEV_TOPK_EXACT_PATH == 0


@pytest.mark.parametrize("kind,schedule,final_k", [("bloom", (1, 40, 24), 32), ("node", (1, 100, 80), 80)])
def test_decode_without_materialised_candidates_equals_the_materialised_path(kind, schedule, final_k):
    """The fast path (mask kernel leaves allow bits, top-k reads the logits through them) must give the same
    beams, bit for bit, as the path that writes the masked candidates and selects from them."""
    cfg = _config1(B=3, matcher_kind=kind, schedule=schedule, final_k=final_k)
    n = cfg["B"] * final_k
    outs = []
    for separate in (True, False):
        dec, api = _make_gpu_decoder(cfg, separate_cand=separate, residual_bf16=True)
        assert (dec.allow_bits is None) == separate
        dec.reset(); dec.decode()
        torch.cuda.synchronize()
        fin = dec.L & 1
        assert dec.d_status.item() & ~api.DEV_TOPK_EXACT_PATH == 0
        outs.append((dec.score[fin][:n].clone(), dec.key[fin][:n].clone(), dec.node[fin][:n].clone(),
                     dec.parents[:, :n].clone()))
    assert torch.equal(outs[0][0].view(torch.int32), outs[1][0].view(torch.int32))
    assert torch.equal(outs[0][1], outs[1][1]) and torch.equal(outs[0][2], outs[1][2])
    assert torch.equal(outs[0][3], outs[1][3])
