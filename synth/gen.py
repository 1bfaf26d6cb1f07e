"""Seeded generators for the decode-step workloads.

Every array that the oracle and the CUDA path must agree on starts here.  The
shapes and distributions follow the paper's evaluation set-up (Section 3.2,
Section 3.3, Section 6.1): thousands of beams per request, SIDs of 3-4 tokens,
encoder K/V shared by every beam of a request, a sparse trie below level 1.

Nothing in this file belongs to the method: it draws numbers, rounds them to
bf16, and de-duplicates SID tuples.  Index structures, hashes and scores are
built separately by each side.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

BASE_SEED = 260800938


def seed_for(config: int, variant: int = 0) -> int:
    """Seed convention: base + 1000 * config + variant."""
    return BASE_SEED + 1000 * int(config) + int(variant)


def rng_for(config: int, variant: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed_for(config, variant)))


# --------------------------------------------------------------------------
# bf16 <-> fp32 (format conversion, round-to-nearest-even)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (RNE) and return the 16-bit patterns as uint16."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to the fp32 values they denote."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32)
            << np.uint32(16)).view(np.float32)


def normal_f32(rng: np.random.Generator, shape, std: float = 1.0) -> np.ndarray:
    return (rng.standard_normal(shape, dtype=np.float32) * np.float32(std)).astype(np.float32)


def normal_bf16(rng: np.random.Generator, shape, std: float = 1.0) -> np.ndarray:
    """N(0, std^2) rounded to bf16; returned as uint16 bit patterns."""
    return f32_to_bf16_bits(normal_f32(rng, shape, std))


# --------------------------------------------------------------------------
# catalog / eligibility
# --------------------------------------------------------------------------
def catalog(rng: np.random.Generator, n_sids: int, V: int, L: int) -> np.ndarray:
    """`n_sids` distinct SIDs, uniform over V**L, as int32 [n_sids, L].

    Rows come back in lexicographic order so that the result does not depend on
    the rejection order.  Requires V**L >= n_sids.
    """
    space = V ** L
    if n_sids > space:
        raise ValueError("catalog larger than the SID space")
    have = np.empty(0, dtype=np.int64)
    while have.size < n_sids:
        need = n_sids - have.size
        draw = rng.integers(0, space, size=int(need * 1.1) + 16, dtype=np.int64)
        have = np.unique(np.concatenate([have, draw]))
    if have.size > n_sids:
        keep = rng.choice(have.size, size=n_sids, replace=False)
        have = np.sort(have[keep])
    sids = np.empty((n_sids, L), dtype=np.int32)
    rest = have.copy()
    for j in range(L - 1, -1, -1):
        sids[:, j] = (rest % V).astype(np.int32)
        rest //= V
    return sids


def eligible_subset(rng: np.random.Generator, n_sids: int, fraction: float) -> np.ndarray:
    """Boolean [n_sids]: exactly round(fraction * n_sids) SIDs marked eligible."""
    k = int(round(fraction * n_sids))
    mask = np.zeros(n_sids, dtype=bool)
    mask[rng.choice(n_sids, size=k, replace=False)] = True
    return mask


def beam_prefixes_from_sids(rng: np.random.Generator, sids: np.ndarray, depth: int,
                            count: int) -> np.ndarray:
    """`count` distinct length-`depth` prefixes of the given SIDs, int32 [count, depth].

    Used to place beams on real trie prefixes: the caller passes the SIDs that
    are eligible for a request, so every returned prefix is catalog-valid and
    has an eligible descendant.  If fewer distinct prefixes exist, all of them
    are returned (the caller pads with dead beams).
    """
    pref = np.unique(sids[:, :depth], axis=0)
    if pref.shape[0] > count:
        keep = np.sort(rng.choice(pref.shape[0], size=count, replace=False))
        pref = pref[keep]
    return pref.astype(np.int32)


def descending_scores(rng: np.random.Generator, count: int, depth: int) -> np.ndarray:
    """Beam scores as a finished top-k leaves them: sorted, non-positive, fp32."""
    s = -np.abs(rng.standard_normal(count)) * max(depth, 1)
    return np.sort(s)[::-1].astype(np.float32)


# --------------------------------------------------------------------------
# log-probabilities and parent indices
# --------------------------------------------------------------------------
def logp_rows(rng: np.random.Generator, R: int, V: int, logit_std: float = 3.0,
              chunk: int = 4096) -> np.ndarray:
    """fp32 [R, V]: log-softmax of N(0, logit_std^2) logits, one row per beam."""
    out = np.empty((R, V), dtype=np.float32)
    for lo in range(0, R, chunk):
        hi = min(R, lo + chunk)
        z = rng.standard_normal((hi - lo, V)) * logit_std
        z -= z.max(axis=1, keepdims=True)
        z -= np.log(np.exp(z).sum(axis=1, keepdims=True))
        out[lo:hi] = z.astype(np.float32)
    return out


def uniform_parents(rng: np.random.Generator, B: int, M_prev: int, M: int) -> np.ndarray:
    """int32 [B*M]: for every new beam row, a parent index uniform in [0, M_prev)."""
    return rng.integers(0, M_prev, size=B * M, dtype=np.int32)


# --------------------------------------------------------------------------
# decoder weights
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class DecoderShape:
    n_layers: int
    d_model: int
    n_heads: int
    d_head: int
    d_ffn: int
    d_enc: int
    V: int
    L: int

    @property
    def d_attn(self) -> int:
        return self.n_heads * self.d_head


def decoder_weights(rng: np.random.Generator, shp: DecoderShape, std: float = 0.02,
                    as_bf16: bool = True) -> dict:
    """Random-init decoder parameters, N(0, std^2); LayerNorm gain 1, bias 0.

    Linear weights are stored [out_features, in_features].  With `as_bf16` the
    values are rounded to bf16 and returned as fp32 holding exactly those
    values, so both sides start from identical numbers.
    """
    def lin(o, i):
        w = normal_f32(rng, (o, i), std)
        return bf16_bits_to_f32(f32_to_bf16_bits(w)) if as_bf16 else w

    d, da = shp.d_model, shp.d_attn
    w = {
        "embed": lin(shp.V + 1, d),          # row V is BOS
        "pos": lin(shp.L, d),
        "lnf_g": np.ones(d, np.float32), "lnf_b": np.zeros(d, np.float32),
        "w_out": lin(shp.V, d),
        "layers": [],
    }
    for _ in range(shp.n_layers):
        w["layers"].append({
            "ln1_g": np.ones(d, np.float32), "ln1_b": np.zeros(d, np.float32),
            "w_qkv": lin(3 * da, d),
            "w_o": lin(d, da),
            "ln2_g": np.ones(d, np.float32), "ln2_b": np.zeros(d, np.float32),
            "w_qc": lin(da, d),
            "w_kc": lin(da, shp.d_enc),
            "w_vc": lin(da, shp.d_enc),
            "w_oc": lin(d, da),
            "ln3_g": np.ones(d, np.float32), "ln3_b": np.zeros(d, np.float32),
            "w_1": lin(shp.d_ffn, d),
            "w_2": lin(d, shp.d_ffn),
        })
    return w


# --------------------------------------------------------------------------
# ads targeting rows (inputs of the per-node matcher form, Sections 4.2 / 4.3)
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class TargetingLayout:
    """Bit layout of the packed attribute mask and the size of the Bloom rows.

    attributes: (first_bit, n_values) per low-cardinality attribute, packed into W_bm 64-bit words.
    Locations are the high-cardinality attribute: each of `n_locations` ids owns `bits_per_location`
    fixed positions of a (64 * W_bl)-bit Bloom row (the positions are drawn once, here: turning a
    location string into its row is outside the decode path, the rows arrive pre-built).
    """
    W_bm: int = 7
    W_bl: int = 4
    attributes: tuple = ((0, 200), (200, 8), (208, 3), (211, 40), (251, 12), (263, 100), (363, 60))
    n_locations: int = 5000
    bits_per_location: int = 3


def _set_bits(rows: np.ndarray, row_ids: np.ndarray, bit_ids: np.ndarray) -> None:
    np.bitwise_or.at(rows, (row_ids, bit_ids >> 6), np.uint64(1) << (bit_ids & 63).astype(np.uint64))


def location_rows(rng: np.random.Generator, layout: TargetingLayout) -> np.ndarray:
    """uint64 [n_locations, W_bl]: the Bloom row bloom(l) of every location id."""
    rows = np.zeros((layout.n_locations, layout.W_bl), dtype=np.uint64)
    pos = rng.integers(0, 64 * layout.W_bl, size=(layout.n_locations, layout.bits_per_location))
    ids = np.repeat(np.arange(layout.n_locations), layout.bits_per_location)
    _set_bits(rows, ids, pos.reshape(-1))
    return rows


def ads_for_sids(rng: np.random.Generator, n_sids: int, layout: TargetingLayout, loc_rows: np.ndarray):
    """Synthetic ads under every SID (1 / 2 / 11 ads per SID at p50 / p90 / p99, like the paper's index).

    Returns (ad_sid int64 [n_ads], ad_bitmask uint64 [n_ads, W_bm], ad_bloom uint64 [n_ads, W_bl]).
    An ad allows, per attribute, either every value (probability 0.5) or 1-3 random values, and
    targets 1-4 random locations.
    """
    u = rng.random(n_sids)
    n_ads = np.where(u < 0.55, 1, np.where(u < 0.90, 2, np.where(u < 0.985, rng.integers(3, 9, n_sids),
                                                                   rng.integers(9, 25, n_sids))))
    ad_sid = np.repeat(np.arange(n_sids, dtype=np.int64), n_ads)
    total = ad_sid.shape[0]
    bm = np.zeros((total, layout.W_bm), dtype=np.uint64)
    for first, n_values in layout.attributes:
        everything = rng.random(total) < 0.5
        ids = np.nonzero(everything)[0]
        _set_bits(bm, np.repeat(ids, n_values), np.tile(first + np.arange(n_values), ids.shape[0]))
        ids = np.nonzero(~everything)[0]
        for _ in range(3):
            keep = rng.random(ids.shape[0]) < (1.0 if _ == 0 else 0.5)
            _set_bits(bm, ids[keep], first + rng.integers(0, n_values, size=int(keep.sum())))
    bl = np.zeros((total, layout.W_bl), dtype=np.uint64)
    for _ in range(4):
        keep = rng.random(total) < (1.0 if _ == 0 else 0.4)
        loc = rng.integers(0, layout.n_locations, size=int(keep.sum()))
        bl[keep] |= loc_rows[loc]
    return ad_sid, bm, bl


def request_attributes(rng: np.random.Generator, B: int, layout: TargetingLayout, loc_rows: np.ndarray,
                       n_loc: int = 64):
    """Per request: one observed value per attribute -> uint64 [B, W_bm]; n_loc user locations ->
    uint64 [B, n_loc, W_bl] (their Bloom rows) and the location ids int64 [B, n_loc]."""
    ubm = np.zeros((B, layout.W_bm), dtype=np.uint64)
    for first, n_values in layout.attributes:
        _set_bits(ubm, np.arange(B), first + rng.integers(0, n_values, size=B))
    loc = rng.integers(0, layout.n_locations, size=(B, n_loc))
    return ubm, loc_rows[loc], loc
