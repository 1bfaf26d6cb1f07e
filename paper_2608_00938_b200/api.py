"""ctypes binding of the C ABI declared in include/grace.h.

Functions take torch CUDA tensors (device memory and the current stream come
from torch; nothing else does) or numpy arrays for the host-side index
builders.  Names match the C entry points.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgrace_b200.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2608_00938_b200.build` "
        "(there is no fallback path)")

lib = C.CDLL(LIB_PATH)

GRACE_OK = 0
DEV_BAD_INDEX, DEV_NAN, DEV_TIMEOUT, DEV_TOPK_EXACT_PATH = 1, 2, 4, 8
MATCH_NONE, MATCH_NODE_BITMASK, MATCH_PREFIX_BLOOM = 0, 1, 2
MAX_LAYERS, MAX_STEPS = 16, 8

_vp, _i32, _i64, _f32, _sz = C.c_void_p, C.c_int, C.c_int64, C.c_float, C.c_size_t


class TrieStruct(C.Structure):
    _fields_ = [("V", C.c_int32), ("L", C.c_int32), ("num_nodes", C.c_int64),
                ("num_internal", C.c_int64), ("child_bits", _vp), ("child_base", _vp)]


class MatcherStruct(C.Structure):
    _fields_ = [("kind", C.c_int32), ("bloom_log2_bits", C.c_int32), ("bloom_hashes", C.c_int32),
                ("reserved", C.c_int32), ("words_per_request", C.c_int64), ("bits", _vp)]


class GtmIndexStruct(C.Structure):
    _fields_ = [("V", C.c_int32), ("L", C.c_int32), ("W_bm", C.c_int32), ("W_bl", C.c_int32), ("N_loc", C.c_int32),
                ("reserved", C.c_int32), ("num_nodes", C.c_int64), ("num_entries", C.c_int64),
                ("node_offsets", _vp), ("csr_child_nodes", _vp), ("csr_tokens", _vp), ("bitmask_index", _vp),
                ("bloom_index", _vp), ("bitmask_table", _vp), ("bloom_table", _vp), ("user_bitmask", _vp),
                ("user_blooms", _vp), ("part_offsets", _vp)]


class LayerStruct(C.Structure):
    _fields_ = [(n, _vp) for n in (
        "ln1_g", "ln1_b", "ln2_g", "ln2_b", "ln3_g", "ln3_b",
        "w_qkv", "w_o", "w_qc", "w_oc", "w_1", "w_2",
        "k_cross", "v_cross", "k_cache", "v_cache",
        "cs_qkv", "cb_qkv", "cs_qc", "cb_qc", "cs_1", "cb_1", "qkv_slabs")]


class DecoderStruct(C.Structure):
    _fields_ = [
        ("B", C.c_int32), ("n_layers", C.c_int32), ("d_model", C.c_int32), ("H", C.c_int32),
        ("d_h", C.c_int32), ("d_ffn", C.c_int32), ("V", C.c_int32), ("L", C.c_int32),
        ("T_ctx", C.c_int32),
        ("beam_sizes", C.c_int32 * (MAX_STEPS + 1)),
        ("R_max", C.c_int64),
        ("ln_eps", C.c_float),
        ("layers", LayerStruct * MAX_LAYERS),
        ("embed", _vp), ("pos", _vp), ("lnf_g", _vp), ("lnf_b", _vp), ("w_out", _vp),
        ("trie", TrieStruct), ("matcher", MatcherStruct),
        ("token", _vp * 2), ("score", _vp * 2), ("node", _vp * 2), ("key", _vp * 2),
        ("parents", _vp), ("out_flat", _vp),
        ("x", _vp), ("x_bf16", _vp), ("h", _vp), ("qkv", _vp), ("attn", _vp), ("logp", _vp), ("row_lse", _vp), ("cand", _vp), ("allow_bits", _vp), ("masked_from_step", C.c_int32),
        ("logits_allowed_only", C.c_int32), ("lse_part", _vp), ("row_affine", _vp), ("cs_out", _vp), ("cb_out", _vp),
        ("topk_ws", _vp), ("topk_ws_bytes", C.c_size_t),
        ("d_status", _vp),
    ]


def _sig(name, restype, argtypes):
    fn = getattr(lib, name)
    fn.restype = restype
    fn.argtypes = argtypes
    return fn


_status_string = _sig("grace_status_string", C.c_char_p, [_i32])
_version = _sig("grace_version", _i32, [])
_built_for_sm = _sig("grace_built_for_sm", _i32, [])
_trie_count_nodes = _sig("grace_trie_count_nodes", _i32, [_vp, _i64, _i32, _i32, _vp])
_trie_build_dense = _sig("grace_trie_build_dense", _i32, [_vp, _i64, _i32, _i32, _vp, _vp])
_node_bitmask_build = _sig("grace_node_bitmask_build", _i32, [_vp, _i64, _i32, _i32, _vp, _vp])
_fold_layer_norm = _sig("grace_fold_layer_norm", _i32, [_vp, _vp, _vp, _i64, _i64, _vp, _vp, _vp])
_centre_rows = _sig("grace_centre_rows", _i32, [_vp, _i64, _i64, _vp])
_centre_outputs = _sig("grace_centre_outputs", _i32, [_vp, _i64, _i64, _vp])
_f32_to_bf16 = _sig("grace_f32_to_bf16", _i32, [_vp, _i64, _vp])
_bloom_build = _sig("grace_bloom_build", _i32, [_vp, _i64, _i32, _i32, _vp, _i32, _i32, _vp])
_trie_walk = _sig("grace_trie_walk", _i32, [_vp, _vp, _i32, _i32, _i64, _vp, _i32, _vp])
_cross_attn = _sig("grace_cross_attn", _i32, [_vp, _i64, _vp, _vp, _i64, _i64, _i64, _vp, _i64, _vp,
                                             _i32, _i32, _i32, _i32, _i32, _f32, _vp, _vp])
_cross_attn_varlen = _sig("grace_cross_attn_varlen", _i32, [_vp, _i64, _vp, _vp, _i64, _i64, _i64, _vp, _i64, _vp, _vp,
                                                           _i32, _i32, _i32, _i32, _i32, _f32, _vp, _vp])
_self_attn = _sig("grace_self_attn", _i32, [_vp, _i64, _vp, _vp, _vp, _vp, _vp, _i64,
                                           _i32, _i32, _i32, _i32, _i64, _f32, _vp, _vp])
_self_attn_inplace = _sig("grace_self_attn_inplace", _i32, [_vp, _i64, _i64, _vp, _vp, _vp, _i64,
                                                           _i32, _i32, _i32, _i32, _i64, _f32, _vp, _vp])
_gtm_mask = _sig("grace_gtm_mask", _i32, [_vp, _vp, _vp, _vp, C.POINTER(TrieStruct), C.POINTER(MatcherStruct),
                                         _vp, _vp, _i32, _i32, _i32, _i32, _vp, _vp])
_gtm_mask_logits = _sig("grace_gtm_mask_logits", _i32, [_vp, _vp, _vp, _vp, _vp, C.POINTER(TrieStruct),
                                                       C.POINTER(MatcherStruct), _vp, _vp, _i32, _i32, _i32, _i32, _vp, _vp])
_gtm_index_build = _sig("grace_gtm_index_build", _i32, [_vp, _i64, _i32, _i32, _vp, _i64, _vp, _i32, _vp, _i32,
                                                       _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp])
_gtm_index_build_kway = _sig("grace_gtm_index_build_kway", _i32,
                             [_vp, _i64, _i32, _i32, _vp, _i64, _vp, _i32, _vp, _i32, _vp, C.c_double, _i32,
                              _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp])
_beam_topk_masked = _sig("grace_beam_topk_masked", _i32, [_vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp,
                                                         _vp, C.c_size_t, _vp, _vp])
_linear_f32_lse = _sig("grace_linear_f32_lse", _i32, [_vp, _i64, _vp, _i64, _vp, _i64, _vp, _i32, _i32, _i32, _vp])
_gtm_mask_logits_parts = _sig("grace_gtm_mask_logits_parts", _i32,
                              [_vp, _vp, _vp, _vp, _vp, C.POINTER(TrieStruct), C.POINTER(MatcherStruct), _vp, _vp,
                               _i32, _i32, _i32, _i32, _vp, _i32, _vp, _vp])
_row_stats_bf16 = _sig("grace_row_stats_bf16", _i32, [_vp, _i32, _i32, _f32, _vp, _vp])
_linear_folded_ln = _sig("grace_linear_folded_ln", _i32, [_vp, _i64, _vp, _i64, _vp, _vp, _vp, _vp, _vp, _i64, _vp,
                                                         _i32, _i32, _i32, _i32, _vp])
_linear_layer_norm = _sig("grace_linear_layer_norm", _i32, [_vp, _i64, _vp, _i64, _f32, _vp, _vp, _vp, _vp, _vp, _i64, _vp,
                                                           _i32, _i32, _i32, _i32, _vp])
_linear_logits_allowed = _sig("grace_linear_logits_allowed", _i32, [_vp, _i64, _vp, _i64, _f32, _vp, _vp, _vp, _vp, _vp, _i64,
                                                                   _vp, _i32, _i32, _i32, _vp])
_gtm_allow_bits = _sig("grace_gtm_allow_bits", _i32, [_vp, _vp, C.POINTER(TrieStruct), C.POINTER(MatcherStruct), _vp,
                                                     _i32, _i32, _i32, _i32, _vp, _vp])
_row_lse_from_parts = _sig("grace_row_lse_from_parts", _i32, [_vp, _i32, _vp, C.POINTER(TrieStruct), _vp, _i32, _vp])
_wait_timeouts = _sig("grace_wait_timeouts", _i32, [])
_stream_l2_persist = _sig("grace_stream_l2_persist", _i32, [_vp, _vp, C.c_size_t, C.c_float])
_selftest_bounded_wait = _sig("grace_selftest_bounded_wait", _i32, [_vp])
_gtm_lookup = _sig("grace_gtm_lookup", _i32, [_vp, _vp, _vp, C.POINTER(GtmIndexStruct), _vp, _vp, _i32, _i32, _vp, _vp])
_beam_update_csr = _sig("grace_beam_update_csr", _i32, [_vp, _vp, _vp, _vp, _vp, C.POINTER(GtmIndexStruct), _vp, _vp,
                                                       _i32, _i32, _i32, _i32, _vp, _vp])
_topk_ws = _sig("grace_beam_topk_workspace_bytes", _sz, [_i32, _i64, _i32])
_beam_topk = _sig("grace_beam_topk", _i32, [_vp, _i32, _i64, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _sz, _vp, _vp])
_beam_topk_static = _sig("grace_beam_topk_static", _i32, [_vp, _i32, _i64, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp])
_beam_topk_static_max = _sig("grace_beam_topk_static_max_requests", _i32, [])
_beam_update = _sig("grace_beam_update", _i32, [_vp, _vp, _vp, _vp, _vp, C.POINTER(TrieStruct), _vp, _vp,
                                               _i32, _i32, _i32, _i32, _vp, _vp])
_linear = _sig("grace_linear", _i32, [_vp, _i64, _vp, _i64, _vp, _vp, _i64, _vp, _i32, _i32, _i32, _i32, _vp])
_linear_add_bf16 = _sig("grace_linear_add_bf16", _i32, [_vp, _i64, _vp, _i64, _vp, _i64, _i32, _i32, _i32, _vp])
_layer_norm_bf16 = _sig("grace_layer_norm_bf16", _i32, [_vp, _vp, _vp, _vp, _i32, _i32, _f32, _vp])
_embed_bf16 = _sig("grace_embed_bf16", _i32, [_vp, _vp, _vp, _vp, _i32, _i32, _i32, _vp, _vp])
_layer_norm = _sig("grace_layer_norm", _i32, [_vp, _vp, _vp, _vp, _i32, _i32, _f32, _vp])
_embed = _sig("grace_embed", _i32, [_vp, _vp, _vp, _vp, _i32, _i32, _i32, _vp, _vp])
_log_softmax = _sig("grace_log_softmax", _i32, [_vp, _i32, _i32, _vp])
_decoder_validate = _sig("grace_decoder_validate", _i32, [C.POINTER(DecoderStruct)])
_decode_step = _sig("grace_decode_step", _i32, [C.POINTER(DecoderStruct), _i32, _vp])
_decode_begin = _sig("grace_decode_begin", _i32, [C.POINTER(DecoderStruct), _vp])
_launch_count = _sig("grace_kernel_launch_count", C.c_uint64, [])


class GraceError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {_status_string(code).decode()} ({code})")


def _check(code: int, where: str) -> None:
    if code != GRACE_OK:
        raise GraceError(code, where)


def _dp(t):
    """Device pointer of a torch tensor (None -> NULL)."""
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "expected a contiguous CUDA tensor"
    return t.data_ptr()


def _hp(a, dtype):
    assert isinstance(a, np.ndarray) and a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    return a.ctypes.data


def _stream():
    import torch
    return torch.cuda.current_stream().cuda_stream


def version() -> int:
    return _version()


def built_for_sm() -> int:
    return _built_for_sm()


# ----------------------------------------------------------------------------
# host-side index builders (numpy in, numpy out)
# ----------------------------------------------------------------------------
def grace_trie_count_nodes(sids: np.ndarray, V: int) -> np.ndarray:
    n, L = sids.shape
    level_start = np.zeros(L + 2, dtype=np.int64)
    _check(_trie_count_nodes(_hp(sids, np.int32), n, V, L, level_start.ctypes.data), "grace_trie_count_nodes")
    return level_start


def grace_trie_build_dense(sids: np.ndarray, V: int):
    """-> (child_bits uint64 [n_internal, V/64], child_base int32 [n_internal], level_start)."""
    n, L = sids.shape
    level_start = grace_trie_count_nodes(sids, V)
    n_int = int(level_start[L])
    bits = np.empty((n_int, V // 64), dtype=np.uint64)
    base = np.empty(n_int, dtype=np.int32)
    _check(_trie_build_dense(_hp(sids, np.int32), n, V, L, bits.ctypes.data, base.ctypes.data),
           "grace_trie_build_dense")
    return bits, base, level_start


def grace_node_bitmask_build(sids: np.ndarray, V: int, eligible: np.ndarray, num_nodes: int) -> np.ndarray:
    n, L = sids.shape
    out = np.empty((num_nodes + 63) // 64, dtype=np.uint64)
    el = np.ascontiguousarray(eligible, dtype=np.uint8)
    _check(_node_bitmask_build(_hp(sids, np.int32), n, V, L, el.ctypes.data, out.ctypes.data),
           "grace_node_bitmask_build")
    return out


def grace_bloom_build(sids: np.ndarray, V: int, eligible: np.ndarray, log2_bits: int, n_hashes: int) -> np.ndarray:
    n, L = sids.shape
    out = np.empty((1 << log2_bits) // 64, dtype=np.uint64)
    el = np.ascontiguousarray(eligible, dtype=np.uint8)
    _check(_bloom_build(_hp(sids, np.int32), n, V, L, el.ctypes.data, log2_bits, n_hashes, out.ctypes.data),
           "grace_bloom_build")
    return out


def grace_fold_layer_norm(w: np.ndarray, gamma: np.ndarray, beta: np.ndarray):
    """Host: (w * gamma as bf16 bits uint16 [N, K], column sums fp32 [N], w @ beta fp32 [N])."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    g = np.ascontiguousarray(gamma, dtype=np.float32)
    b = np.ascontiguousarray(beta, dtype=np.float32)
    N, K = w.shape
    assert g.shape == (K,) and b.shape == (K,)
    wf, cs, cb = np.empty((N, K), np.uint16), np.empty(N, np.float32), np.empty(N, np.float32)
    _check(_fold_layer_norm(w.ctypes.data, g.ctypes.data, b.ctypes.data, N, K, wf.ctypes.data, cs.ctypes.data,
                            cb.ctypes.data), "grace_fold_layer_norm")
    return wf, cs, cb


def grace_centre_rows(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    out = np.empty_like(a)
    _check(_centre_rows(a.ctypes.data, a.shape[0], a.shape[1], out.ctypes.data), "grace_centre_rows")
    return out


def grace_centre_outputs(w: np.ndarray) -> np.ndarray:
    w = np.ascontiguousarray(w, dtype=np.float32)
    out = np.empty_like(w)
    _check(_centre_outputs(w.ctypes.data, w.shape[0], w.shape[1], out.ctypes.data), "grace_centre_outputs")
    return out


def grace_f32_to_bf16(a: np.ndarray) -> np.ndarray:
    """Host: fp32 array -> bf16 bit patterns (uint16, same shape), round to nearest even."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    out = np.empty(a.shape, np.uint16)
    _check(_f32_to_bf16(a.ctypes.data, a.size, out.ctypes.data), "grace_f32_to_bf16")
    return out


def grace_trie_walk(child_bits: np.ndarray, child_base: np.ndarray, V: int, L: int, tokens) -> int:
    tok = np.ascontiguousarray(tokens, dtype=np.int32)
    node = C.c_int32(-2)
    _check(_trie_walk(_hp(child_bits, np.uint64), _hp(child_base, np.int32), V, L, child_bits.shape[0],
                      tok.ctypes.data, tok.shape[0], C.addressof(node)), "grace_trie_walk")
    return node.value


def grace_gtm_index_build(sids: np.ndarray, V: int, ad_sid: np.ndarray, ad_bitmask: np.ndarray, ad_bloom: np.ndarray):
    """Host build of the paper-form index -> dict of numpy arrays (Appendix A field names)."""
    n, L = sids.shape
    num_nodes = int(grace_trie_count_nodes(sids, V)[-1])
    E = num_nodes - 1
    W_bm, W_bl = ad_bitmask.shape[1], ad_bloom.shape[1]
    out = dict(node_offsets=np.empty(num_nodes + 1, np.int32), csr_child_nodes=np.empty(E, np.int32),
               csr_tokens=np.empty(E, np.int16), bitmask_index=np.empty(E, np.int32), bloom_index=np.empty(E, np.int32))
    ad_sid = np.ascontiguousarray(ad_sid, dtype=np.int64)
    n_bm, n_bl = C.c_int64(0), C.c_int64(0)

    def call(bm_table, bl_table):
        return _gtm_index_build(_hp(sids, np.int32), n, V, L, ad_sid.ctypes.data, ad_sid.shape[0],
                                _hp(ad_bitmask, np.uint64), W_bm, _hp(ad_bloom, np.uint64), W_bl,
                                out["node_offsets"].ctypes.data, out["csr_child_nodes"].ctypes.data,
                                out["csr_tokens"].ctypes.data, out["bitmask_index"].ctypes.data,
                                out["bloom_index"].ctypes.data, bm_table, C.addressof(n_bm), bl_table, C.addressof(n_bl))
    _check(call(None, None), "grace_gtm_index_build (sizes)")
    out["bitmask_table"] = np.empty((n_bm.value, W_bm), np.uint64)
    out["bloom_table"] = np.empty((n_bl.value, W_bl), np.uint64)
    _check(call(out["bitmask_table"].ctypes.data, out["bloom_table"].ctypes.data), "grace_gtm_index_build")
    out.update(num_nodes=num_nodes, V=V, L=L)
    return out


def grace_gtm_index_build_kway(sids: np.ndarray, V: int, ad_sid: np.ndarray, ad_bitmask: np.ndarray, ad_bloom: np.ndarray,
                               k_level=None, fill_target: float = 0.0, k_max: int = 1):
    """Host build of the index with k-way partitioned rows: static (k_level[l] per node level) or dynamic
    (fill_target, k_max).  Returns the dict of grace_gtm_index_build plus part_offsets; bitmask_index and
    bloom_index are per partition slot."""
    n, L = sids.shape
    num_nodes = int(grace_trie_count_nodes(sids, V)[-1])
    E = num_nodes - 1
    W_bm, W_bl = ad_bitmask.shape[1], ad_bloom.shape[1]
    out = dict(node_offsets=np.empty(num_nodes + 1, np.int32), csr_child_nodes=np.empty(E, np.int32),
               csr_tokens=np.empty(E, np.int16), part_offsets=np.empty(E + 1, np.int32))
    ad_sid = np.ascontiguousarray(ad_sid, dtype=np.int64)
    kl = None if k_level is None else np.ascontiguousarray(k_level, dtype=np.int32)
    assert kl is None or kl.shape[0] == L + 1
    n_parts, n_bm, n_bl = C.c_int64(0), C.c_int64(0), C.c_int64(0)

    def call(pbm, pbl, bm_table, bl_table):
        return _gtm_index_build_kway(_hp(sids, np.int32), n, V, L, ad_sid.ctypes.data, ad_sid.shape[0],
                                     _hp(ad_bitmask, np.uint64), W_bm, _hp(ad_bloom, np.uint64), W_bl,
                                     None if kl is None else kl.ctypes.data, float(fill_target), int(k_max),
                                     out["node_offsets"].ctypes.data, out["csr_child_nodes"].ctypes.data,
                                     out["csr_tokens"].ctypes.data, out["part_offsets"].ctypes.data, pbm, pbl,
                                     C.addressof(n_parts), bm_table, C.addressof(n_bm), bl_table, C.addressof(n_bl))
    _check(call(None, None, None, None), "grace_gtm_index_build_kway (sizes)")
    out["bitmask_index"] = np.empty(n_parts.value, np.int32)
    out["bloom_index"] = np.empty(n_parts.value, np.int32)
    out["bitmask_table"] = np.empty((n_bm.value, W_bm), np.uint64)
    out["bloom_table"] = np.empty((n_bl.value, W_bl), np.uint64)
    _check(call(out["bitmask_index"].ctypes.data, out["bloom_index"].ctypes.data, out["bitmask_table"].ctypes.data,
                out["bloom_table"].ctypes.data), "grace_gtm_index_build_kway")
    out.update(num_nodes=num_nodes, V=V, L=L)
    return out


def make_gtm_index(host_index: dict, user_bitmask: np.ndarray, user_blooms: np.ndarray, device="cuda:0") -> GtmIndexStruct:
    """Upload a host index (from grace_gtm_index_build) and the per-request rows; returns the C struct."""
    import torch

    def up(a):
        if a.dtype == np.uint64:
            a = a.view(np.int64)
        return torch.from_numpy(np.ascontiguousarray(a)).to(device)
    keep = {k: up(host_index[k]) for k in ("node_offsets", "csr_child_nodes", "csr_tokens", "bitmask_index",
                                           "bloom_index", "bitmask_table", "bloom_table")}
    keep["user_bitmask"], keep["user_blooms"] = up(user_bitmask), up(user_blooms)
    if host_index.get("part_offsets") is not None:          # k-way partitioned rows: the index arrays are per slot
        keep["part_offsets"] = up(host_index["part_offsets"])
    s = GtmIndexStruct(host_index["V"], host_index["L"], user_bitmask.shape[1], host_index["bloom_table"].shape[1],
                       user_blooms.shape[1], 0, host_index["num_nodes"], host_index["num_nodes"] - 1,
                       *[keep[k].data_ptr() for k in ("node_offsets", "csr_child_nodes", "csr_tokens", "bitmask_index",
                                                      "bloom_index", "bitmask_table", "bloom_table", "user_bitmask",
                                                      "user_blooms")],
                       keep["part_offsets"].data_ptr() if "part_offsets" in keep else None)
    s._keepalive = keep
    return s


def grace_beam_topk_masked(logits, allow_bits, row_score, row_lse, B: int, M: int, K: int, out_score, out_flat, out_parent,
                           out_token, ws, d_status=None):
    """Top-k over candidates that are never materialised (see grace_beam_topk_masked in grace.h)."""
    V = logits.shape[-1]
    _check(_beam_topk_masked(_dp(logits), _dp(allow_bits), _dp(row_score), _dp(row_lse), B, M, V, K, _dp(out_score),
                             _dp(out_flat), _dp(out_parent), _dp(out_token), _dp(ws), ws.numel() * ws.element_size(),
                             _dp(d_status), _stream()), "grace_beam_topk_masked")


def grace_linear_f32_lse(x, w, y, lse_part):
    """y fp32 [M, N] = x @ w.T and lse_part fp32 [M, N // 256, 2] = per-tile (maximum, sum of e^(y - maximum))."""
    M, K = x.shape
    N = w.shape[0]
    _check(_linear_f32_lse(x.data_ptr(), x.stride(0), w.data_ptr(), w.stride(0), _dp(y), y.stride(0), _dp(lse_part), M, N, K,
                           _stream()), "grace_linear_f32_lse")
    return y, lse_part


def grace_gtm_mask_logits_parts(logits, row_lse, beam_score, beam_node, beam_key, trie, matcher, cand, allow_bits, B: int,
                                M: int, prefix_len: int, lse_part, d_status=None):
    """grace_gtm_mask_logits with the per-tile log-sum-exp partials of grace_linear_f32_lse."""
    V = logits.shape[-1]
    _check(_gtm_mask_logits_parts(_dp(logits), _dp(row_lse), _dp(beam_score), _dp(beam_node), _dp(beam_key), C.byref(trie),
                                  C.byref(matcher), _dp(cand), _dp(allow_bits), B, M, V, prefix_len, _dp(lse_part),
                                  lse_part.shape[1], _dp(d_status), _stream()), "grace_gtm_mask_logits_parts")


def grace_row_stats_bf16(x, row_affine, eps: float = 1e-5):
    """row_affine fp32 [R, 2] = (rstd, -rstd * mean) of the bf16 rows of x."""
    R, D = x.shape
    _check(_row_stats_bf16(_dp(x), R, D, eps, _dp(row_affine), _stream()), "grace_row_stats_bf16")
    return row_affine


def grace_linear_folded_ln(x, w_folded, row_affine, col_sum, col_bias, y, relu: bool = False, lse_part=None):
    """y = row_affine[:, :1] * (x @ w_folded.T) + row_affine[:, 1:] * col_sum + col_bias  (LayerNorm folded into
    the GEMM); y bf16 or fp32.  col_sum None: the rows of x have zero mean and the middle term is dropped."""
    import torch
    M, K = x.shape
    N = w_folded.shape[0]
    f32 = y.dtype == torch.float32
    _check(_linear_folded_ln(x.data_ptr(), x.stride(0), w_folded.data_ptr(), w_folded.stride(0), _dp(row_affine),
                             _dp(col_sum), _dp(col_bias), None if f32 else _dp(y), _dp(y) if f32 else None, y.stride(0),
                             _dp(lse_part), M, N, K, int(relu), _stream()), "grace_linear_folded_ln")
    return y


def grace_linear_layer_norm(x, w_folded, eps: float, row_affine, col_sum, col_bias, y, relu: bool = False, lse_part=None):
    """LayerNorm over the rows of x (statistics with eps) and the GEMM behind it in one call: the result of
    grace_row_stats_bf16 + grace_linear_folded_ln.  row_affine: fp32 [M, 2] scratch (used only when the
    statistics cannot be formed inside the GEMM kernel)."""
    import torch
    M, K = x.shape
    N = w_folded.shape[0]
    f32 = y.dtype == torch.float32
    _check(_linear_layer_norm(x.data_ptr(), x.stride(0), w_folded.data_ptr(), w_folded.stride(0), float(eps),
                              _dp(row_affine), _dp(col_sum), _dp(col_bias), None if f32 else _dp(y),
                              _dp(y) if f32 else None, y.stride(0), _dp(lse_part), M, N, K, int(relu), _stream()),
           "grace_linear_layer_norm")
    return y


def grace_linear_logits_allowed(x, w, allow_bits, y, lse_part, eps: float = 0.0, row_affine=None, col_sum=None,
                                col_bias=None):
    """fp32 logits GEMM that stores only the allowed elements of y (bits [M, N/64] int64) and the log-sum-exp
    partials of all of them; row_affine (fp32 [M, 2] scratch) given: a LayerNorm with eps folded in front."""
    M, K = x.shape
    N = w.shape[0]
    _check(_linear_logits_allowed(x.data_ptr(), x.stride(0), w.data_ptr(), w.stride(0), float(eps), _dp(row_affine),
                                  _dp(col_sum), _dp(col_bias), _dp(allow_bits), _dp(y), y.stride(0), _dp(lse_part),
                                  M, N, K, _stream()), "grace_linear_logits_allowed")
    return y


def grace_gtm_allow_bits(beam_node, beam_key, trie: TrieStruct, matcher: MatcherStruct, allow_bits, B: int, M: int,
                         prefix_len: int, d_status=None):
    """allow_bits [B*M, V/64] = catalog-valid children AND matcher, from the beam state alone."""
    _check(_gtm_allow_bits(_dp(beam_node), _dp(beam_key), C.byref(trie), C.byref(matcher), _dp(allow_bits), B, M,
                           trie.V, prefix_len, _dp(d_status), _stream()), "grace_gtm_allow_bits")
    return allow_bits


def grace_row_lse_from_parts(lse_part, beam_node, trie: TrieStruct, row_lse):
    """row_lse [R] from the logits GEMM's per-tile partials [R, n_parts, 2]; 0 for dead rows."""
    R, n_parts = lse_part.shape[0], lse_part.shape[1]
    _check(_row_lse_from_parts(_dp(lse_part), n_parts, _dp(beam_node), C.byref(trie), _dp(row_lse), R, _stream()),
           "grace_row_lse_from_parts")
    return row_lse


def grace_stream_l2_persist(t=None, fraction: float = 0.5) -> None:
    """Keep `fraction` of tensor `t` resident in L2 for kernels launched on the current stream from now on
    (None clears the window)."""
    if t is None:
        _check(_stream_l2_persist(_stream(), None, 0, 0.0), "grace_stream_l2_persist")
    else:
        _check(_stream_l2_persist(_stream(), t.data_ptr(), t.numel() * t.element_size(), fraction),
               "grace_stream_l2_persist")


def grace_wait_timeouts() -> int:
    """Bounded device waits that gave up since the previous call (0 in normal operation)."""
    return int(_wait_timeouts())


def grace_selftest_bounded_wait() -> int:
    """Runs the bounded-wait self-test; returns the status code (TIMEOUT = the wait gave up as designed)."""
    return int(_selftest_bounded_wait(_stream()))


def grace_gtm_lookup(logp, beam_score, beam_node, index: GtmIndexStruct, cand, allow_bits, B: int, M: int,
                     d_status=None):
    _check(_gtm_lookup(_dp(logp), _dp(beam_score), _dp(beam_node), C.byref(index), _dp(cand), _dp(allow_bits), B, M,
                       _dp(d_status), _stream()), "grace_gtm_lookup")


def grace_beam_update_csr(parent, token, score, prev_node, prev_key, index: GtmIndexStruct, new_node, new_key,
                          B: int, K: int, M_prev: int, prefix_len: int, d_status=None):
    _check(_beam_update_csr(_dp(parent), _dp(token), _dp(score), _dp(prev_node), _dp(prev_key), C.byref(index),
                            _dp(new_node), _dp(new_key), B, K, M_prev, prefix_len, _dp(d_status), _stream()),
           "grace_beam_update_csr")


def make_trie(child_bits_dev, child_base_dev, V: int, L: int, num_nodes: int) -> TrieStruct:
    trie = TrieStruct(V, L, num_nodes, child_bits_dev.shape[0], _dp(child_bits_dev), _dp(child_base_dev))
    trie._keepalive = (child_bits_dev, child_base_dev)      # the struct only holds raw pointers
    return trie


def make_matcher(kind: int, bits_dev=None, log2_bits: int = 0, n_hashes: int = 0) -> MatcherStruct:
    words = 0 if bits_dev is None else bits_dev.shape[-1]
    matcher = MatcherStruct(kind, log2_bits, n_hashes, 0, words, _dp(bits_dev))
    matcher._keepalive = bits_dev
    return matcher


# ----------------------------------------------------------------------------
# device ops (torch CUDA tensors; bf16 tensors are torch.bfloat16)
# ----------------------------------------------------------------------------
def grace_cross_attn(q, k, v, out, scale: float, lse=None, d_status=None):
    """q/out [B*M, H, d] (or [B, M, H, d]) bf16; k/v [B, H, T, d] bf16 (any strides with unit last)."""
    B, H, T, d = k.shape
    q2 = q.reshape(-1, H, d)
    o2 = out.reshape(-1, H, d)
    M = q2.shape[0] // B
    assert k.stride() == v.stride() and k.stride(3) == 1
    _check(_cross_attn(q2.data_ptr(), q2.stride(0), k.data_ptr(), v.data_ptr(), k.stride(0), k.stride(1),
                       k.stride(2), o2.data_ptr(), o2.stride(0), _dp(lse), B, M, H, d, T, scale,
                       _dp(d_status), _stream()), "grace_cross_attn")
    return out


def grace_cross_attn_varlen(q, k, v, out, enc_len, scale: float, lse=None, d_status=None):
    """grace_cross_attn with a per-request number of valid encoder positions: enc_len int32 [B] on the device."""
    B, H, T, d = k.shape
    q2 = q.reshape(-1, H, d)
    o2 = out.reshape(-1, H, d)
    M = q2.shape[0] // B
    assert k.stride() == v.stride() and k.stride(3) == 1 and enc_len.element_size() == 4 and enc_len.numel() == B
    _check(_cross_attn_varlen(q2.data_ptr(), q2.stride(0), k.data_ptr(), v.data_ptr(), k.stride(0), k.stride(1),
                              k.stride(2), o2.data_ptr(), o2.stride(0), _dp(lse), _dp(enc_len), B, M, H, d, T, scale,
                              _dp(d_status), _stream()), "grace_cross_attn_varlen")
    return out


def grace_self_attn(qkv, k_cache, v_cache, parents, beam_sizes, out, B: int, t: int, scale: float,
                    d_status=None):
    """qkv [R, 3, H, d]; caches [L, R_max, H, d]; parents int32 [L, R_max]; out [R, H, d]."""
    R, three, H, d = qkv.shape
    bs = np.ascontiguousarray(beam_sizes[: t + 1], dtype=np.int32)
    _check(_self_attn(_dp(qkv), qkv.stride(0), _dp(k_cache), _dp(v_cache), _dp(parents), bs.ctypes.data,
                      _dp(out), out.stride(0), B, t, H, d, k_cache.shape[1], scale, _dp(d_status), _stream()),
           "grace_self_attn")
    return out


def grace_self_attn_inplace(qkv_slabs, parents, beam_sizes, out, B: int, t: int, scale: float, d_status=None):
    """qkv_slabs [L, R_max, 3, H, d]: slab j is the QKV projection of step j and, in its K and V thirds, the
    cache; parents int32 [L, R_max]; out [R, H, d].  Nothing but `out` is written."""
    L, R_max, three, H, d = qkv_slabs.shape
    bs = np.ascontiguousarray(beam_sizes[: t + 1], dtype=np.int32)
    _check(_self_attn_inplace(_dp(qkv_slabs), qkv_slabs.stride(1), qkv_slabs.stride(0), _dp(parents), bs.ctypes.data,
                              _dp(out), out.stride(0), B, t, H, d, R_max, scale, _dp(d_status), _stream()),
           "grace_self_attn_inplace")
    return out


def grace_gtm_mask(logp, beam_score, beam_node, beam_key, trie: TrieStruct, matcher: MatcherStruct,
                   cand, allow_bits, B: int, M: int, prefix_len: int, d_status=None):
    V = logp.shape[-1]
    _check(_gtm_mask(_dp(logp), _dp(beam_score), _dp(beam_node), _dp(beam_key), C.byref(trie), C.byref(matcher),
                     _dp(cand), _dp(allow_bits), B, M, V, prefix_len, _dp(d_status), _stream()), "grace_gtm_mask")


def grace_gtm_mask_logits(logits, row_lse, beam_score, beam_node, beam_key, trie: TrieStruct, matcher: MatcherStruct,
                          cand, allow_bits, B: int, M: int, prefix_len: int, d_status=None):
    """Fused log-softmax + CD/GTM mask + score add on raw logits [R, V] (V <= 2048)."""
    V = logits.shape[-1]
    _check(_gtm_mask_logits(_dp(logits), _dp(row_lse), _dp(beam_score), _dp(beam_node), _dp(beam_key), C.byref(trie),
                            C.byref(matcher), _dp(cand), _dp(allow_bits), B, M, V, prefix_len, _dp(d_status),
                            _stream()), "grace_gtm_mask_logits")


def grace_beam_topk_workspace_bytes(B: int, N: int, K: int) -> int:
    return _topk_ws(B, N, K)


def grace_beam_topk(cand, K: int, V: int, out_score, out_flat, out_parent, out_token, ws, d_status=None):
    """cand fp32 [B, N]; outputs [B, K]; ws: uint8 CUDA tensor of workspace_bytes."""
    B, N = cand.shape
    _check(_beam_topk(_dp(cand), B, N, K, V, _dp(out_score), _dp(out_flat), _dp(out_parent), _dp(out_token),
                      _dp(ws), ws.numel() * ws.element_size(), _dp(d_status), _stream()), "grace_beam_topk")


def grace_beam_topk_static_max_requests() -> int:
    return _beam_topk_static_max()


def grace_beam_topk_static(cand, K: int, V: int, out_score, out_flat, out_parent, out_token, d_status=None):
    """grace_beam_topk without a caller workspace: the scratch is a fixed array inside the library.

    For callers that cannot allocate device memory at this point (buffers-only plug-ins, hot paths
    on which allocation is forbidden).  At most grace_beam_topk_static_max_requests() requests per
    call; calls on one device share the scratch and must not overlap on the GPU.  The first call on
    a device should happen outside stream capture.
    """
    B, N = cand.shape
    _check(_beam_topk_static(_dp(cand), B, N, K, V, _dp(out_score), _dp(out_flat), _dp(out_parent), _dp(out_token),
                             _dp(d_status), _stream()), "grace_beam_topk_static")


def grace_beam_update(parent, token, score, prev_node, prev_key, trie: TrieStruct, new_node, new_key,
                      B: int, K: int, M_prev: int, prefix_len: int, d_status=None):
    _check(_beam_update(_dp(parent), _dp(token), _dp(score), _dp(prev_node), _dp(prev_key), C.byref(trie),
                        _dp(new_node), _dp(new_key), B, K, M_prev, prefix_len, _dp(d_status), _stream()),
           "grace_beam_update")


def grace_linear(x, w, y, residual=None, relu: bool = False):
    """y = act(x @ w.T) (+ residual); x [M, K] bf16, w [N, K] bf16, y [M, N] bf16 or fp32."""
    import torch
    M, K = x.shape
    N = w.shape[0]
    yb, yf = (_dp(y), None) if y.dtype == torch.bfloat16 else (None, _dp(y))
    _check(_linear(x.data_ptr(), x.stride(0), w.data_ptr(), w.stride(0), yb, yf, y.stride(0),
                   _dp(residual), M, N, K, int(relu), _stream()), "grace_linear")
    return y


def grace_linear_add_bf16(x, w, y):
    """y (bf16 [M, N], in place) += x @ w.T."""
    M, K = x.shape
    N = w.shape[0]
    _check(_linear_add_bf16(x.data_ptr(), x.stride(0), w.data_ptr(), w.stride(0), _dp(y), y.stride(0), M, N, K, _stream()),
           "grace_linear_add_bf16")
    return y


def grace_layer_norm(x, gamma, beta, out, eps: float = 1e-5):
    """x fp32 or bf16 [R, D] -> out bf16."""
    import torch
    R, D = x.shape
    if x.dtype == torch.bfloat16:
        _check(_layer_norm_bf16(_dp(x), _dp(gamma), _dp(beta), _dp(out), R, D, eps, _stream()), "grace_layer_norm_bf16")
        return out
    _check(_layer_norm(_dp(x), _dp(gamma), _dp(beta), _dp(out), R, D, eps, _stream()), "grace_layer_norm")
    return out


def grace_embed(token, embed, pos, x, d_status=None):
    """x fp32 or bf16 [R, D] = embed[token] + pos."""
    import torch
    R, D = x.shape
    if x.dtype == torch.bfloat16:
        _check(_embed_bf16(_dp(token), _dp(embed), _dp(pos), _dp(x), R, D, embed.shape[0], _dp(d_status), _stream()),
               "grace_embed_bf16")
        return x
    _check(_embed(_dp(token), _dp(embed), _dp(pos), _dp(x), R, D, embed.shape[0], _dp(d_status), _stream()),
           "grace_embed")
    return x


def grace_log_softmax(logits):
    R, V = logits.shape
    _check(_log_softmax(_dp(logits), R, V, _stream()), "grace_log_softmax")
    return logits


def grace_decoder_validate(dec: DecoderStruct) -> int:
    return _decoder_validate(C.byref(dec))


def grace_kernel_launch_count() -> int:
    return int(_launch_count())


def grace_decode_begin(dec: DecoderStruct):
    _check(_decode_begin(C.byref(dec), _stream()), "grace_decode_begin")


def grace_decode_step(dec: DecoderStruct, t: int):
    _check(_decode_step(C.byref(dec), t, _stream()), "grace_decode_step")
