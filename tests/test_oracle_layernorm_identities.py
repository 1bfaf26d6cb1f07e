"""Two identities of a pre-LayerNorm decoder that the product path relies on, checked on the oracle alone (fp64):

  * every consumer of the residual stream is a LayerNorm, and LayerNorm does not see a per-row shift, so centring
    everything that is added into the stream (embedding and position rows; the output projections over their
    output index) leaves every log-probability unchanged;
  * LayerNorm(x) @ w^T = rstd * (x @ (w * gamma)^T) - rstd * mean * colsum(w * gamma) + beta @ w^T.
"""
import copy

import numpy as np

import synth
from oracle import decoder as D


def _setup(seed=3):
    rng = synth.rng_for(1, 500 + seed)
    shp = synth.DecoderShape(2, 64, 4, 16, 128, 48, 32, 3)
    w = synth.decoder_weights(rng, shp, std=0.2, as_bf16=False)
    for holder, names in [(w, ("lnf",))] + [(lw, ("ln1", "ln2", "ln3")) for lw in w["layers"]]:
        for n in names:
            holder[n + "_g"] = (1.0 + 0.3 * synth.normal_f32(rng, shp.d_model)).astype(np.float64)
            holder[n + "_b"] = (0.4 * synth.normal_f32(rng, shp.d_model)).astype(np.float64)
    w["embed"] = np.asarray(w["embed"], np.float64) + 1.5          # rows with a mean
    enc = synth.normal_f32(rng, (2, 10, 48)).astype(np.float64)
    return rng, shp, w, enc


def _log_probs(w, shp, enc, steps=3, M=5):
    B = enc.shape[0]
    rng = synth.rng_for(1, 777)
    sizes = [1] + [M] * (steps - 1)
    state = D.DecoderState(shp, B, sizes)
    ckv = D.cross_kv(w, shp, enc)
    out = []
    tokens = np.full(B, shp.V)
    for t in range(steps):
        out.append(D.decoder_forward(w, shp, state, ckv, tokens, t, B))
        if t + 1 < steps:
            state.parents[t + 1] = synth.uniform_parents(rng, B, sizes[t], sizes[t + 1]).astype(np.int32)
            tokens = rng.integers(0, shp.V, B * sizes[t + 1])
    return out


def test_centring_the_producers_of_the_stream_changes_no_log_probability():
    _, shp, w, enc = _setup()
    ref = _log_probs(w, shp, enc)
    c = copy.deepcopy(w)
    c["embed"] = c["embed"] - c["embed"].mean(axis=1, keepdims=True)
    c["pos"] = np.asarray(c["pos"], np.float64) - np.asarray(c["pos"], np.float64).mean(axis=1, keepdims=True)
    for lw in c["layers"]:
        for name in ("w_o", "w_oc", "w_2"):                      # [d_model, K]: centre over the output index
            a = np.asarray(lw[name], np.float64)
            lw[name] = a - a.mean(axis=0, keepdims=True)
    got = _log_probs(c, shp, enc)
    for a, b in zip(ref, got):
        np.testing.assert_allclose(b, a, rtol=0, atol=1e-9)
    # and it is not vacuous: the uncentred stream does carry a mean, and centring something else does change the result
    assert abs(np.asarray(w["embed"]).mean()) > 1.0
    bad = copy.deepcopy(w)
    bad["layers"][0]["w_1"] = np.asarray(bad["layers"][0]["w_1"], np.float64) - np.asarray(bad["layers"][0]["w_1"]).mean(axis=0, keepdims=True)
    assert np.abs(_log_probs(bad, shp, enc)[1] - ref[1]).max() > 1e-6


def test_layer_norm_folds_into_the_matrix_behind_it():
    rng, shp, w, _ = _setup(4)
    x = synth.normal_f32(rng, (7, shp.d_model)).astype(np.float64) * 2.0 + 0.7
    lw = w["layers"][0]
    g, b, wt = np.asarray(lw["ln1_g"], np.float64), np.asarray(lw["ln1_b"], np.float64), np.asarray(lw["w_qkv"], np.float64)
    ref = D.layer_norm(x, g, b) @ wt.T
    mean = x.mean(axis=1, keepdims=True)
    rstd = 1.0 / np.sqrt(x.var(axis=1, keepdims=True) + 1e-5)
    wf = wt * g[None, :]
    got = rstd * (x @ wf.T) - rstd * mean * wf.sum(axis=1)[None, :] + (wt @ b)[None, :]
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-10)
    # with centred rows the middle term is zero
    xc = x - mean
    np.testing.assert_allclose(rstd * (xc @ wf.T) + (wt @ b)[None, :], ref, rtol=0, atol=1e-10)
