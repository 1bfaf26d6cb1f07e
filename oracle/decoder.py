"""Oracle: decoder forward pass and GTM-constrained beam search.  Test infrastructure.

Sections 3.1-3.3: an autoregressive loop over SID positions; each step runs
the decoder on the current beam rows, turns logits into log-probabilities,
applies the CD + GTM mask, adds the prefix score, selects the top M_{t+1}
candidates per request and carries their parent, token, score and trie node
forward.  Cross-attention K/V are projected once per request from the encoder
output and shared by all beams (Section 3.2).

PARITY UNPINNED for the layer internals: the paper states the number of
layers, heads and the head size but not the arrangement inside a layer.  The
reading used: pre-LayerNorm (eps 1e-5) residual blocks in the order
self-attention, cross-attention, ReLU feed-forward; no linear biases; a learned
position vector per SID position added to the token embedding; input table row
V is the start token; final LayerNorm and an untied output head; log-softmax
over the whole vocabulary at temperature 1.
"""
from __future__ import annotations

import numpy as np

from . import attention, gtm, topk

U64 = np.uint64


def layer_norm(x, g, b, eps=1e-5):
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * g + b


def log_softmax(z):
    z = z - z.max(axis=-1, keepdims=True)
    return z - np.log(np.exp(z).sum(axis=-1, keepdims=True))


def cross_kv(weights, shp, enc, dtype=np.float64):
    """Per layer: K_c, V_c [B, H, T_ctx, d_h] from the encoder output [B, T_ctx, d_enc]."""
    enc = np.asarray(enc, dtype=dtype)
    B, T, _ = enc.shape
    out = []
    for lw in weights["layers"]:
        k = (enc @ lw["w_kc"].astype(dtype).T).reshape(B, T, shp.n_heads, shp.d_head)
        v = (enc @ lw["w_vc"].astype(dtype).T).reshape(B, T, shp.n_heads, shp.d_head)
        out.append((k.transpose(0, 2, 1, 3).copy(), v.transpose(0, 2, 1, 3).copy()))
    return out


class DecoderState:
    """Self-attention caches (one pair per layer) and the parent arrays."""

    def __init__(self, shp, B, beam_sizes, dtype=np.float64):
        R_max = B * max(beam_sizes)
        self.k = [np.zeros((shp.L, R_max, shp.n_heads, shp.d_head), dtype) for _ in range(shp.n_layers)]
        self.v = [np.zeros((shp.L, R_max, shp.n_heads, shp.d_head), dtype) for _ in range(shp.n_layers)]
        self.parents = [None] * shp.L          # parents[j], j >= 1
        self.beam_sizes = list(beam_sizes)


def decoder_forward(weights, shp, state, ckv, tokens, t, B, dtype=np.float64, trace=None):
    """Log-probabilities [B * M_t, V] for the rows whose input tokens are `tokens`.

    `tokens` [B * M_t]: the token chosen at step t-1 (V = start token at t = 0).
    Writes slab t of every layer's cache in `state`.
    """
    H, dh = shp.n_heads, shp.d_head
    scale = 1.0 / np.sqrt(dh)
    M_t = state.beam_sizes[t]
    R = B * M_t
    W = lambda a: np.asarray(a, dtype=dtype)
    x = W(weights["embed"])[np.asarray(tokens)] + W(weights["pos"])[t]
    for li, lw in enumerate(weights["layers"]):
        h = layer_norm(x, W(lw["ln1_g"]), W(lw["ln1_b"]))
        qkv = (h @ W(lw["w_qkv"]).T).reshape(R, 3, H, dh)
        o, kc, vc = attention.self_attn(qkv, state.k[li], state.v[li], state.parents,
                                        state.beam_sizes, t, B, scale)
        state.k[li], state.v[li] = kc.astype(dtype), vc.astype(dtype)
        x = x + o.reshape(R, H * dh).astype(dtype) @ W(lw["w_o"]).T
        h = layer_norm(x, W(lw["ln2_g"]), W(lw["ln2_b"]))
        qc = (h @ W(lw["w_qc"]).T).reshape(B, M_t, H, dh)
        oc, _ = attention.cross_attn(qc, ckv[li][0], ckv[li][1], scale)
        x = x + oc.reshape(R, H * dh).astype(dtype) @ W(lw["w_oc"]).T
        h = layer_norm(x, W(lw["ln3_g"]), W(lw["ln3_b"]))
        x = x + np.maximum(h @ W(lw["w_1"]).T, 0) @ W(lw["w_2"]).T
        if trace is not None:
            trace.append(x.copy())
    logits = layer_norm(x, W(weights["lnf_g"]), W(weights["lnf_b"])) @ W(weights["w_out"]).T
    return log_softmax(logits)


def beam_search(weights, shp, enc, trie, matcher, schedule, final_k, dtype=np.float64,
                record=None):
    """GTM-constrained beam search.  schedule = (M_0 = 1, M_1, ..., M_{L-1}); the
    last step selects `final_k` SIDs.

    Returns dict(sids int [B, final_k, L], score f32 [B, final_k], valid bool [B, final_k]).
    `record`, if a list, receives one dict per step with every intermediate.
    """
    enc = np.asarray(enc)
    B = enc.shape[0]
    L, V = shp.L, shp.V
    assert len(schedule) == L and schedule[0] == 1
    state = DecoderState(shp, B, schedule, dtype)
    ckv = cross_kv(weights, shp, enc, dtype)
    tokens = np.full(B, V, dtype=np.int64)                 # start token
    score = np.zeros(B, dtype=np.float32)
    node = np.zeros(B, dtype=np.int32)                     # root
    key = np.zeros(B, dtype=U64)
    history = []                                           # (parent, token) per step
    for t in range(L):
        M_t = schedule[t]
        K = schedule[t + 1] if t + 1 < L else final_k
        logp = decoder_forward(weights, shp, state, ckv, tokens, t, B, dtype).astype(np.float32)
        cand, allow, child = gtm.gtm_mask(logp, score, node, key, t, trie, matcher, B, M_t)
        sc, flat, par, tok = topk.beam_topk(cand.reshape(B, M_t * V), K, V)
        new_node, new_key = topk.update_beam_state(trie, par, tok, sc, node, key, t, M_t)
        if record is not None:
            record.append(dict(t=t, tokens=tokens.copy(), score=score.copy(), node=node.copy(),
                               key=key.copy(), logp=logp, cand=cand, allow=allow,
                               out_score=sc, out_flat=flat, out_parent=par, out_token=tok,
                               new_node=new_node, new_key=new_key))
        history.append((par, tok))
        if t + 1 < L:
            state.parents[t + 1] = par.reshape(-1).astype(np.int32)
        tokens, score, node, key = tok.reshape(-1).astype(np.int64), sc.reshape(-1), new_node, new_key
    # read the SIDs back by following parents
    sids = np.zeros((B, final_k, L), dtype=np.int64)
    for b in range(B):
        for i in range(final_k):
            idx = i
            for t in range(L - 1, -1, -1):
                par, tok = history[t]
                sids[b, i, t] = tok[b, idx]
                idx = par[b, idx]
    return dict(sids=sids, score=sc, valid=~np.isneginf(sc), node=node.reshape(B, final_k))
