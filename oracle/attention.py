"""Oracle: the two attentions of the decode step, in fp64.  Test infrastructure.

Cross-attention (Section 5.1, Appendix B): the M beams of request b are M query
positions against that request's one copy of K[b, h], V[b, h]; the reshape is
layout only, so the result is textbook scaled-dot-product attention per row.

Self-attention (Sections 5.2, 5.3): row r at step t attends to its own prefix
0..t (current token included), nothing else; the prefix of a row is found by
following parent indices (equivalently the block table P with
P_new[i, j] = P[p_i, j] for j < t and a fresh block for position t).
"""
from __future__ import annotations

import numpy as np


def _softmax(x: np.ndarray, axis: int = -1) -> np.ndarray:
    x = x - x.max(axis=axis, keepdims=True)
    e = np.exp(x)
    return e / e.sum(axis=axis, keepdims=True)


# ---------------------------------------------------------------------------
# cross-attention
# ---------------------------------------------------------------------------
def cross_attn(q, k, v, scale, return_probs: bool = False):
    """q [B, M, H, d], k/v [B, H, T, d] -> out [B, M, H, d] (and lse [B, M, H]).

    out[b, m, h] = softmax_t(q[b, m, h] . k[b, h, t] * scale) @ v[b, h].
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    B, M, H, d = q.shape
    out = np.empty((B, M, H, d), dtype=np.float64)
    lse = np.empty((B, M, H), dtype=np.float64)
    probs = [] if return_probs else None
    for b in range(B):
        for h in range(H):
            s = (q[b, :, h, :] @ k[b, h].T) * scale            # [M, T]
            p = _softmax(s, axis=1)
            out[b, :, h, :] = p @ v[b, h]
            smax = s.max(axis=1)
            lse[b, :, h] = smax + np.log(np.exp(s - smax[:, None]).sum(axis=1))
            if return_probs:
                probs.append(p)
    if return_probs:
        return out, lse, probs
    return out, lse


def cross_attn_varlen(q, k, v, enc_len, scale):
    """Cross-attention over padded encoder outputs: request b attends to its first enc_len[b] positions only
    (an extension: Section 3.2 fixes the encoder length per batch).  A request without any position gets
    zero output and lse = -inf.  Written as the definition: the plain cross-attention of every request on
    its own, truncated K / V."""
    q = np.asarray(q, dtype=np.float64)
    B, M, H, d = q.shape
    out = np.zeros((B, M, H, d), dtype=np.float64)
    lse = np.full((B, M, H), -np.inf, dtype=np.float64)
    for b in range(B):
        n = int(enc_len[b])
        if n > 0:
            o, l = cross_attn(q[b:b + 1], np.asarray(k)[b:b + 1, :, :n], np.asarray(v)[b:b + 1, :, :n], scale)
            out[b], lse[b] = o[0], l[0]
    return out, lse


def cross_attn_row(q_row, k_bh, v_bh, scale):
    """One (beam row, head): q_row [d], k_bh/v_bh [T, d] -> [d]."""
    s = (np.asarray(k_bh, np.float64) @ np.asarray(q_row, np.float64)) * scale
    return _softmax(s) @ np.asarray(v_bh, np.float64)


# ---------------------------------------------------------------------------
# self-attention over the parent-addressed cache
# ---------------------------------------------------------------------------
def ancestors(parents, beam_sizes, t: int, b: int, m: int):
    """Rows (one per step 0..t) that hold the prefix of beam m of request b.

    parents[j] (j = 1..t) is int [B * M_j]: the index, inside request b's
    step-(j-1) beam, of the row that row (b, m) of step j extends.
    Returns global row indices a[0..t], a[j] = b * M_j + local_j.
    """
    rows = [0] * (t + 1)
    local = m
    for j in range(t, -1, -1):
        rows[j] = b * beam_sizes[j] + local
        if j > 0:
            local = int(parents[j][b * beam_sizes[j] + local])
    return rows


def self_attn(qkv, k_cache, v_cache, parents, beam_sizes, t: int, B: int, scale):
    """One step of fused self-attention.

    qkv      [R, 3, H, d]          projection output for the R = B * M_t rows
    k_cache  [L, R_max, H, d]      slabs 0..t-1 filled by earlier steps
    v_cache  same
    Writes slab t (rows 0..R-1) of copies of the caches and returns
    (out [R, H, d], k_cache', v_cache').
    """
    qkv = np.asarray(qkv, dtype=np.float64)
    kc = np.array(k_cache, dtype=np.float64, copy=True)
    vc = np.array(v_cache, dtype=np.float64, copy=True)
    M_t = beam_sizes[t]
    R = B * M_t
    assert qkv.shape[0] == R
    H, d = qkv.shape[2], qkv.shape[3]
    kc[t, :R] = qkv[:, 1]
    vc[t, :R] = qkv[:, 2]
    out = np.empty((R, H, d), dtype=np.float64)
    for b in range(B):
        for m in range(M_t):
            r = b * M_t + m
            rows = ancestors(parents, beam_sizes, t, b, m)
            keys = np.stack([kc[j, rows[j]] for j in range(t + 1)])     # [t+1, H, d]
            vals = np.stack([vc[j, rows[j]] for j in range(t + 1)])
            for h in range(H):
                s = (keys[:, h, :] @ qkv[r, 0, h, :]) * scale          # [t+1]
                out[r, h] = _softmax(s) @ vals[:, h, :]
    return out, kc, vc


def self_attn_row(qkv_row, kc, vc, parents, beam_sizes, t: int, b: int, m: int, scale):
    """One row of `self_attn`, reading slabs < t from the caches and slab t from
    the row's own k, v.  qkv_row [3, H, d] -> [H, d]."""
    qkv_row = np.asarray(qkv_row, dtype=np.float64)
    rows = ancestors(parents, beam_sizes, t, b, m)
    keys = [np.asarray(kc[j, rows[j]], np.float64) for j in range(t)] + [qkv_row[1]]
    vals = [np.asarray(vc[j, rows[j]], np.float64) for j in range(t)] + [qkv_row[2]]
    keys, vals = np.stack(keys), np.stack(vals)
    H = qkv_row.shape[1]
    out = np.empty_like(qkv_row[0])
    for h in range(H):
        out[h] = _softmax((keys[:, h, :] @ qkv_row[0, h, :]) * scale) @ vals[:, h, :]
    return out


# ---- equivalent formulations used to pin the parent walk -----------------------
def block_table(parents, beam_sizes, t: int, B: int) -> np.ndarray:
    """Section 5.3 block table P [B * M_t, t + 1], built by the copy rule
    P_new[i, j] = P[p_i, j] (j < step), P_new[i, step] = fresh block i."""
    P = np.arange(B * beam_sizes[0], dtype=np.int64)[:, None]
    for step in range(1, t + 1):
        M_prev, M = beam_sizes[step - 1], beam_sizes[step]
        P_new = np.empty((B * M, step + 1), dtype=np.int64)
        for b in range(B):
            for m in range(M):
                i = b * M + m
                p_i = b * M_prev + int(parents[step][i])
                P_new[i, :step] = P[p_i, :step]
                P_new[i, step] = i
        P = P_new
    return P


def self_attn_block_table(qkv, k_cache, v_cache, parents, beam_sizes, t, B, scale):
    """Same result through the block table instead of the parent walk."""
    qkv = np.asarray(qkv, dtype=np.float64)
    kc = np.array(k_cache, dtype=np.float64, copy=True)
    vc = np.array(v_cache, dtype=np.float64, copy=True)
    R = B * beam_sizes[t]
    kc[t, :R], vc[t, :R] = qkv[:, 1], qkv[:, 2]
    P = block_table(parents, beam_sizes, t, B)
    H, d = qkv.shape[2], qkv.shape[3]
    out = np.empty((R, H, d), dtype=np.float64)
    for r in range(R):
        keys = np.stack([kc[j, P[r, j]] for j in range(t + 1)])
        vals = np.stack([vc[j, P[r, j]] for j in range(t + 1)])
        for h in range(H):
            out[r, h] = _softmax((keys[:, h, :] @ qkv[r, 0, h, :]) * scale) @ vals[:, h, :]
    return out


def dense_reordered_cache(cache, parents, beam_sizes, t: int, B: int) -> np.ndarray:
    """The dense alternative of Section 3.3: after every step copy each selected
    parent's prefix KV into the child's row.  Returns [B * M_t, t, H, d]."""
    cache = np.asarray(cache, dtype=np.float64)
    dense = np.empty((B * beam_sizes[0], 0) + cache.shape[2:], dtype=np.float64)
    for step in range(1, t + 1):
        M_prev, M = beam_sizes[step - 1], beam_sizes[step]
        # previous rows gain their own step-(step-1) entry, then children copy it
        prev_full = np.concatenate([dense, cache[step - 1, :B * M_prev][:, None]], axis=1)
        new = np.empty((B * M,) + prev_full.shape[1:], dtype=np.float64)
        for b in range(B):
            for m in range(M):
                new[b * M + m] = prev_full[b * M_prev + int(parents[step][b * M + m])]
        dense = new
    return dense


def self_attn_dense(qkv, k_cache, v_cache, parents, beam_sizes, t, B, scale):
    """Same result on a densely re-ordered cache (no indirection at attention time)."""
    qkv = np.asarray(qkv, dtype=np.float64)
    dk = dense_reordered_cache(k_cache, parents, beam_sizes, t, B)
    dv = dense_reordered_cache(v_cache, parents, beam_sizes, t, B)
    R, H, d = qkv.shape[0], qkv.shape[2], qkv.shape[3]
    out = np.empty((R, H, d), dtype=np.float64)
    for r in range(R):
        keys = np.concatenate([dk[r], qkv[r, 1][None]], axis=0)
        vals = np.concatenate([dv[r], qkv[r, 2][None]], axis=0)
        for h in range(H):
            out[r, h] = _softmax((keys[:, h, :] @ qkv[r, 0, h, :]) * scale) @ vals[:, h, :]
    return out


def coalesced_tile_attn(q_rows, k_rows, v_rows, scale):
    """Section 5.2 formulation: G rows in one tile with a block-diagonal mask.

    q_rows [G, d], k_rows/v_rows [G, T, d].  Scores form a [G, G*T] tile; entries
    whose key belongs to another row are set to -inf before the softmax.
    """
    q_rows = np.asarray(q_rows, np.float64)
    G, T, d = np.asarray(k_rows).shape
    k_flat = np.asarray(k_rows, np.float64).reshape(G * T, d)
    v_flat = np.asarray(v_rows, np.float64).reshape(G * T, d)
    s = (q_rows @ k_flat.T) * scale
    mask = np.kron(np.eye(G), np.ones((1, T)))             # the matrix printed in Section 5.2
    s = np.where(mask == 1, s, -np.inf)
    return _softmax(s, axis=1) @ v_flat, mask
