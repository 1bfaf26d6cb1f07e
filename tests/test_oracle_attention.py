"""Pins for oracle.attention: closed forms, brute force, the paper's printed
block-diagonal example and layout identity.  CPU only."""
import math
import os

import numpy as np
import pytest
from scipy.special import logsumexp

import synth
from oracle import attention as A


def _pure_python_attention(q, K, V, scale):
    """Independent restatement with python floats and loops."""
    s = [scale * sum(q[i] * K[t][i] for i in range(len(q))) for t in range(len(K))]
    m = max(s)
    e = [math.exp(x - m) for x in s]
    z = sum(e)
    return [sum(e[t] / z * V[t][i] for t in range(len(K))) for i in range(len(V[0]))]


def test_hand_computed_case():
    # scores [0, ln 3] -> probabilities [1/4, 3/4]; values [8], [4] -> 2 + 3 = 5
    q = np.array([[[[1.0]]]])
    k = np.array([[[[0.0], [math.log(3.0)]]]])
    v = np.array([[[[8.0], [4.0]]]])
    out, lse = A.cross_attn(q, k, v, 1.0)
    assert out[0, 0, 0, 0] == pytest.approx(5.0, abs=1e-13)
    assert lse[0, 0, 0] == pytest.approx(math.log(4.0), abs=1e-13)


def test_cross_attn_matches_pure_python_on_ragged_shape():
    rng = np.random.default_rng(1)
    B, M, H, d, T = 2, 5, 3, 7, 11          # all different: a transposed operand cannot pass
    q = rng.standard_normal((B, M, H, d))
    k = rng.standard_normal((B, H, T, d))
    v = rng.standard_normal((B, H, T, d))
    out, lse, probs = A.cross_attn(q, k, v, 0.37, return_probs=True)
    for p in probs:
        np.testing.assert_allclose(p.sum(axis=1), 1.0, atol=1e-12)
    for b in range(B):
        for m in range(M):
            for h in range(H):
                ref = _pure_python_attention(list(q[b, m, h]), k[b, h].tolist(), v[b, h].tolist(), 0.37)
                np.testing.assert_allclose(out[b, m, h], ref, atol=1e-12)
                np.testing.assert_allclose(A.cross_attn_row(q[b, m, h], k[b, h], v[b, h], 0.37), ref, atol=1e-12)
                assert lse[b, m, h] == pytest.approx(logsumexp(0.37 * k[b, h] @ q[b, m, h]), abs=1e-12)


def test_cross_attn_closed_forms():
    rng = np.random.default_rng(2)
    B, M, H, d, T = 2, 4, 2, 8, 6
    q = rng.standard_normal((B, M, H, d))
    v = rng.standard_normal((B, H, T, d))
    # one encoder position: the output is that value row, whatever q is
    out, _ = A.cross_attn(q, rng.standard_normal((B, H, 1, d)), v[:, :, :1], 0.5)
    np.testing.assert_allclose(out, np.broadcast_to(v[:, :, 0][:, None], out.shape), atol=1e-13)
    # identical keys: uniform weights -> mean of the values
    k_same = np.broadcast_to(rng.standard_normal((B, H, 1, d)), (B, H, T, d))
    out, _ = A.cross_attn(q, k_same, v, 0.5)
    np.testing.assert_allclose(out, np.broadcast_to(v.mean(axis=2)[:, None], out.shape), atol=1e-12)
    # permuting encoder positions changes nothing
    k = rng.standard_normal((B, H, T, d))
    perm = rng.permutation(T)
    a, _ = A.cross_attn(q, k, v, 0.5)
    b_, _ = A.cross_attn(q, k[:, :, perm], v[:, :, perm], 0.5)
    np.testing.assert_allclose(a, b_, atol=1e-12)
    # a key that dominates (huge score) selects its value
    k_big = k.copy()
    k_big[:, :, 3] = 0
    q1 = np.ones((B, M, H, d))
    k_big[:, :, 3] = 100.0
    out, _ = A.cross_attn(q1, k_big, v, 1.0)
    np.testing.assert_allclose(out, np.broadcast_to(v[:, :, 3][:, None], out.shape), atol=1e-9)


def test_beam_as_query_layout_identity():
    """Appendix B: view / permute / reshape around SDPA is layout only."""
    rng = np.random.default_rng(3)
    B, M, H, d, T, Tq = 3, 4, 2, 5, 7, 1
    Q = rng.standard_normal((B * M, H, Tq, d))          # beam-major rows r = b*M + m
    k = rng.standard_normal((B, H, T, d))
    v = rng.standard_normal((B, H, T, d))
    # forward chain of Section 5.1
    q = Q.reshape(B, M, H, Tq, d).transpose(0, 2, 1, 3, 4).reshape(B, H, M * Tq, d)
    x = np.empty_like(q)
    for b in range(B):
        for h in range(H):
            s = q[b, h] @ k[b, h].T * 0.3
            p = np.exp(s - s.max(1, keepdims=True))
            x[b, h] = (p / p.sum(1, keepdims=True)) @ v[b, h]
    X = x.reshape(B, H, M, Tq, d).transpose(0, 2, 1, 3, 4).reshape(B * M, H, Tq, d)
    out, _ = A.cross_attn(Q[:, :, 0, :].reshape(B, M, H, d), k, v, 0.3)
    np.testing.assert_allclose(out.reshape(B * M, H, d), X[:, :, 0, :], atol=1e-12)
    # and equals BM unrelated single-query attentions with K/V broadcast per beam
    for r in range(B * M):
        for h in range(H):
            np.testing.assert_allclose(out.reshape(B * M, H, d)[r, h],
                                       A.cross_attn_row(Q[r, h, 0], k[r // M, h], v[r // M, h], 0.3), atol=1e-12)


def _random_self_attn_problem(seed, B, beam_sizes, H, d, L):
    rng = np.random.default_rng(seed)
    t = len(beam_sizes) - 1
    R_max = B * max(beam_sizes)
    kc = np.zeros((L, R_max, H, d))
    vc = np.zeros((L, R_max, H, d))
    parents = [None] * (t + 1)
    for j in range(t):
        kc[j, :B * beam_sizes[j]] = rng.standard_normal((B * beam_sizes[j], H, d))
        vc[j, :B * beam_sizes[j]] = rng.standard_normal((B * beam_sizes[j], H, d))
    for j in range(1, t + 1):
        parents[j] = rng.integers(0, beam_sizes[j - 1], size=B * beam_sizes[j])
    qkv = rng.standard_normal((B * beam_sizes[t], 3, H, d))
    return qkv, kc, vc, parents


@pytest.mark.parametrize("beam_sizes", [(1,), (1, 4), (1, 3, 5), (2, 4, 4, 3), (1, 6, 6, 6, 6)])
def test_parent_walk_equals_block_table_equals_dense_copy(beam_sizes):
    B, H, d, L = 3, 2, 4, 5
    t = len(beam_sizes) - 1
    qkv, kc, vc, parents = _random_self_attn_problem(10 + t, B, list(beam_sizes), H, d, L)
    out, kc2, vc2 = A.self_attn(qkv, kc, vc, parents, list(beam_sizes), t, B, 0.5)
    out_bt = A.self_attn_block_table(qkv, kc, vc, parents, list(beam_sizes), t, B, 0.5)
    out_dense = A.self_attn_dense(qkv, kc, vc, parents, list(beam_sizes), t, B, 0.5)
    assert np.array_equal(out, out_bt)
    assert np.array_equal(out, out_dense)
    # cache write: slab t holds the rows' own k, v; older slabs untouched
    R = B * beam_sizes[t]
    assert np.array_equal(kc2[t, :R], qkv[:, 1]) and np.array_equal(vc2[t, :R], qkv[:, 2])
    assert np.array_equal(kc2[:t], kc[:t]) and np.array_equal(vc2[:t], vc[:t])
    # row-wise form agrees and matches the pure-python restatement
    for r in range(R):
        b, m = divmod(r, beam_sizes[t])
        row = A.self_attn_row(qkv[r], kc, vc, parents, list(beam_sizes), t, b, m, 0.5)
        assert np.array_equal(row, out[r])
        rows = A.ancestors(parents, list(beam_sizes), t, b, m)
        for h in range(H):
            K = [kc2[j, rows[j], h].tolist() for j in range(t + 1)]
            V = [vc2[j, rows[j], h].tolist() for j in range(t + 1)]
            np.testing.assert_allclose(out[r, h], _pure_python_attention(qkv[r, 0, h].tolist(), K, V, 0.5), atol=1e-12)


def test_block_table_copy_rule():
    """P_new[i, j] = P[p_i, j] for j < t (Section 5.3), fresh block at column t."""
    B, sizes = 2, [1, 3, 4]
    parents = [None, np.array([0, 0, 0, 0, 0, 0]), np.array([2, 0, 1, 1, 0, 0, 2, 2])]
    P = A.block_table(parents, sizes, 2, B)
    assert P.shape == (8, 3)
    assert P[:, 2].tolist() == list(range(8))                       # fresh blocks
    assert P[:4, 1].tolist() == [2, 0, 1, 1]                        # request 0: local parents
    assert P[4:, 1].tolist() == [3 + 0, 3 + 0, 3 + 2, 3 + 2]        # request 1: offset by M_1 = 3
    assert P[:4, 0].tolist() == [0] * 4 and P[4:, 0].tolist() == [1] * 4
    for i in range(8):
        assert A.ancestors(parents, sizes, 2, i // 4, i % 4) == P[i].tolist()


def test_first_step_returns_own_value():
    qkv, kc, vc, parents = _random_self_attn_problem(5, 4, [3], 2, 8, 4)
    out, _, _ = A.self_attn(qkv, kc, vc, parents, [3], 0, 4, 0.125)
    np.testing.assert_allclose(out, qkv[:, 2], atol=1e-15)


def test_block_diagonal_example_of_section_5_2(golden_dir):
    rows = [l.split() for l in open(os.path.join(golden_dir, "block_diagonal_g4_t3.txt")) if l[0] in "01"]
    printed = np.array(rows, dtype=float)
    rng = np.random.default_rng(7)
    G, T, d = 4, 3, 6
    q, k, v = rng.standard_normal((G, d)), rng.standard_normal((G, T, d)), rng.standard_normal((G, T, d))
    out, mask = A.coalesced_tile_attn(q, k, v, 0.4)
    assert np.array_equal(mask, printed)
    for g in range(G):                                             # four independent 1 x 3 attentions
        np.testing.assert_allclose(out[g], _pure_python_attention(q[g].tolist(), k[g].tolist(), v[g].tolist(), 0.4), atol=1e-12)


def test_bf16_round_trip_is_rne():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.0e-39, 65504.0, 0.1], dtype=np.float32)
    bits = synth.f32_to_bf16_bits(x)
    back = synth.bf16_bits_to_f32(bits)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7: ties go to the even mantissa (1.0)
    assert back[0] == 1.0 and back[1] == 1.0
    # 1 + 3 * 2^-8 is a tie between 1 + 2^-7 (odd) and 1 + 2^-6 (even)
    assert back[2] == np.float32(1.015625)
    assert back[3] == -2.5
    assert abs(back[6] - 0.1) <= 0.1 * 2 ** -8
    import torch
    assert torch.equal(torch.from_numpy(x).to(torch.bfloat16).float(), torch.from_numpy(back))


def test_cross_attn_with_encoder_lengths_is_attention_over_the_truncated_encoder():
    """`cross_attn_varlen`: pure-Python softmax over each request's first enc_len positions; padding beyond
    them has no influence; a request without positions gets zeros."""
    rng = np.random.default_rng(11)
    B, M, H, d, T = 3, 4, 2, 5, 9
    q, k, v = rng.normal(size=(B, M, H, d)), rng.normal(size=(B, H, T, d)), rng.normal(size=(B, H, T, d))
    enc_len = [9, 4, 0]
    out, lse = A.cross_attn_varlen(q, k, v, enc_len, 0.3)
    k2, v2 = k.copy(), v.copy()
    for b in range(B):
        k2[b, :, enc_len[b]:] = 1e3
        v2[b, :, enc_len[b]:] = -1e3
    out2, _ = A.cross_attn_varlen(q, k2, v2, enc_len, 0.3)
    assert np.array_equal(out, out2)
    for b in range(B):
        for m in range(M):
            for h in range(H):
                n = enc_len[b]
                if n == 0:
                    assert (out[b, m, h] == 0).all() and lse[b, m, h] == -np.inf
                    continue
                s = [0.3 * sum(q[b, m, h, i] * k[b, h, t, i] for i in range(d)) for t in range(n)]
                mx = max(s)
                w = [np.exp(x - mx) for x in s]
                z = sum(w)
                want = [sum(w[t] * v[b, h, t, i] for t in range(n)) / z for i in range(d)]
                np.testing.assert_allclose(out[b, m, h], want, rtol=1e-12, atol=1e-12)
                np.testing.assert_allclose(lse[b, m, h], mx + np.log(z), rtol=1e-12)
