"""Seeded synthetic inputs shared by the CPU oracle and the CUDA path.

This package holds random draws and number-format conversion only: no trie
construction, no hashing, no attention, no masking, no selection.  Both sides
receive the same arrays and do all of the method's arithmetic themselves.
"""
from .gen import (  # noqa: F401
    BASE_SEED,
    seed_for,
    rng_for,
    f32_to_bf16_bits,
    bf16_bits_to_f32,
    normal_bf16,
    normal_f32,
    catalog,
    eligible_subset,
    logp_rows,
    uniform_parents,
    decoder_weights,
    DecoderShape,
    beam_prefixes_from_sids,
    descending_scores,
    TargetingLayout,
    location_rows,
    ads_for_sids,
    request_attributes,
)
