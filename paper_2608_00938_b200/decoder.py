"""Buffer set-up for grace_decode_step: uploads weights and index structures,
allocates the caller-owned state / cache / activation buffers with torch and
fills the C struct.  No arithmetic happens here: every step of the decode path
runs in the library's kernels, and the one-time weight preparation of the
folded-LayerNorm configuration (gain folded into the weights, producers of the
residual stream centred, bf16 conversion) is done by the library's host-side
helpers (grace_fold_layer_norm, grace_centre_rows, grace_centre_outputs,
grace_f32_to_bf16), so a caller of the C ABI gets the same operands."""
from __future__ import annotations

import ctypes as C

import numpy as np
import torch

from . import api


def _bf16_bits(bits: np.ndarray, device) -> torch.Tensor:
    """bf16 bit patterns (uint16) -> device bf16 tensor of the same shape."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


def _bf16(a: np.ndarray, device) -> torch.Tensor:
    return _bf16_bits(api.grace_f32_to_bf16(a), device)


def _f32(a: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device)


class Decoder:
    """Owns the device buffers of one decode loop and the grace_decoder_t that points at them.

    weights: dict as produced by `synth.decoder_weights` (fp32 arrays; matrices are rounded to
    bf16 on upload).  beam_sizes: (M_0 .. M_{L-1}, K_final).  trie_bits / trie_base: host arrays
    from `api.grace_trie_build_dense`.  matcher: (kind, host uint64 [B, words] or None,
    log2_bits, n_hashes).  level_start (optional, from the same trie build): first node id of every level;
    used to decide per step whether masked candidates are written out or read through allow bits.
    """

    def __init__(self, *, n_layers, d_model, n_heads, d_head, d_ffn, V, L, T_ctx, B, beam_sizes, weights,
                 trie_bits, trie_base, num_nodes, matcher=(api.MATCH_NONE, None, 0, 0), device="cuda:0",
                 separate_cand=False, fuse_log_softmax=True, residual_bf16=False, materialize_cand=None,
                 level_start=None, lse_from_gemm=True, fold_layer_norm=None, centre_stream=None,
                 persist_stream_l2=None, kv_in_place=True, logits_allowed_only=False, masked_from_step=None):
        assert len(beam_sizes) == L + 1
        self.device = torch.device(device)
        self.B, self.L, self.V, self.H, self.d_h, self.T_ctx = B, L, V, n_heads, d_head, T_ctx
        self.d_model, self.d_ffn, self.n_layers = d_model, d_ffn, n_layers
        self.beam_sizes = list(beam_sizes)
        HD = n_heads * d_head
        self.R_max = R_max = B * max(beam_sizes)
        dev = self.device
        self._keep = []
        s = api.DecoderStruct()
        s.B, s.n_layers, s.d_model, s.H, s.d_h, s.d_ffn, s.V, s.L, s.T_ctx = (
            B, n_layers, d_model, n_heads, d_head, d_ffn, V, L, T_ctx)
        for i, m in enumerate(beam_sizes):
            s.beam_sizes[i] = m
        s.R_max = R_max
        s.ln_eps = 1e-5
        self.w_kc, self.w_vc, self.k_cross, self.v_cross, self.k_cache, self.v_cache = [], [], [], [], [], []
        self.kv_in_place, self.qkv_slabs = kv_in_place, []
        # LayerNorms folded into the GEMMs behind them (bf16 residual stream): the GEMM reads the raw stream, its
        # weights carry the gain, and its epilogue applies the row statistics (see grace_linear_folded_ln)
        if fold_layer_norm is None:
            fold_layer_norm = residual_bf16 and d_model <= 2048
        assert not fold_layer_norm or residual_bf16
        self.fold_layer_norm = fold_layer_norm
        # Centred stream: every consumer of the residual stream is a LayerNorm, which does not see a per-row
        # shift, so the embedding rows and the projections that add into the stream are centred over the feature
        # axis once, here; the rows then keep zero mean and the folded GEMMs drop their column-sum term.
        if centre_stream is None:
            centre_stream = fold_layer_norm
        assert not centre_stream or fold_layer_norm
        self.centre_stream = centre_stream

        def centred_rows(a):                               # [n, d_model]: each row minus its mean
            return api.grace_centre_rows(a) if centre_stream else a

        def centred_outputs(w):                            # [d_model, K]: minus the mean over the output index
            return api.grace_centre_outputs(w) if centre_stream else w

        def fold(w, gamma, beta):
            """(w * gamma as the bf16 the GEMM will use, column sums of that, beta @ w^T), uploaded."""
            wf, cs, cb = api.grace_fold_layer_norm(w, gamma, beta)
            return _bf16_bits(wf, dev), torch.from_numpy(cs).to(dev), torch.from_numpy(cb).to(dev)

        self.folded = []                                   # per layer: {weight name: (folded weight, column sums, bias)}
        for li, lw in enumerate(weights["layers"]):
            lay = s.layers[li]
            self.folded.append({})
            for name in ("ln1_g", "ln1_b", "ln2_g", "ln2_b", "ln3_g", "ln3_b"):
                t = _f32(lw[name], dev); self._keep.append(t); setattr(lay, name, t.data_ptr())
            for name in ("w_qkv", "w_o", "w_qc", "w_oc", "w_1", "w_2"):
                t = _bf16(centred_outputs(lw[name]) if name in ("w_o", "w_oc", "w_2") else lw[name], dev)
                self._keep.append(t); setattr(lay, name, t.data_ptr())
            if fold_layer_norm:
                for wname, ln, short in (("w_qkv", "ln1", "qkv"), ("w_qc", "ln2", "qc"), ("w_1", "ln3", "1")):
                    wf, cs, cb = fold(lw[wname], lw[ln + "_g"], lw[ln + "_b"])
                    self.folded[li][wname] = (wf, cs, cb)
                    setattr(lay, wname, wf.data_ptr())
                    setattr(lay, "cs_" + short, None if centre_stream else cs.data_ptr())
                    setattr(lay, "cb_" + short, cb.data_ptr())
            self.w_kc.append(_bf16(lw["w_kc"], dev))
            self.w_vc.append(_bf16(lw["w_vc"], dev))
            self.k_cross.append(torch.zeros((B, T_ctx, n_heads, d_head), dtype=torch.bfloat16, device=dev))
            self.v_cross.append(torch.zeros((B, T_ctx, n_heads, d_head), dtype=torch.bfloat16, device=dev))
            lay.k_cross, lay.v_cross = self.k_cross[li].data_ptr(), self.v_cross[li].data_ptr()
            if kv_in_place:
                # the cache is the steps' own QKV projections, kept: nothing is copied into a cache
                self.qkv_slabs.append(torch.zeros((L, R_max, 3, n_heads, d_head), dtype=torch.bfloat16, device=dev))
                lay.qkv_slabs = self.qkv_slabs[li].data_ptr()
            else:
                self.k_cache.append(torch.zeros((L, R_max, n_heads, d_head), dtype=torch.bfloat16, device=dev))
                self.v_cache.append(torch.zeros((L, R_max, n_heads, d_head), dtype=torch.bfloat16, device=dev))
                lay.k_cache, lay.v_cache = self.k_cache[li].data_ptr(), self.v_cache[li].data_ptr()
        self.embed = _bf16(centred_rows(weights["embed"]), dev)
        self.pos = _bf16(centred_rows(weights["pos"]), dev)
        self.lnf_g, self.lnf_b = _f32(weights["lnf_g"], dev), _f32(weights["lnf_b"], dev)
        self.w_out = _bf16(weights["w_out"], dev)
        if fold_layer_norm:
            self.w_out, self.cs_out, self.cb_out = fold(weights["w_out"], weights["lnf_g"], weights["lnf_b"])
            s.cs_out, s.cb_out = None if centre_stream else self.cs_out.data_ptr(), self.cb_out.data_ptr()
        s.embed, s.pos, s.lnf_g, s.lnf_b, s.w_out = (self.embed.data_ptr(), self.pos.data_ptr(),
                                                     self.lnf_g.data_ptr(), self.lnf_b.data_ptr(),
                                                     self.w_out.data_ptr())
        # index structures
        self.trie_bits = torch.from_numpy(trie_bits.view(np.int64)).to(dev)
        self.trie_base = torch.from_numpy(trie_base).to(dev)
        self.trie = api.make_trie(self.trie_bits, self.trie_base, V, L, num_nodes)
        kind, mbits, log2_bits, n_hashes = matcher
        self.matcher_bits = None if mbits is None else torch.from_numpy(
            np.ascontiguousarray(mbits).view(np.int64)).to(dev)
        self.matcher = api.make_matcher(kind, self.matcher_bits, log2_bits, n_hashes)
        s.trie, s.matcher = self.trie, self.matcher
        # beam state
        self.token = [torch.zeros(R_max, dtype=torch.int32, device=dev) for _ in range(2)]
        self.score = [torch.zeros(R_max, dtype=torch.float32, device=dev) for _ in range(2)]
        self.node = [torch.zeros(R_max, dtype=torch.int32, device=dev) for _ in range(2)]
        self.key = [torch.zeros(R_max, dtype=torch.int64, device=dev) for _ in range(2)]
        for i in range(2):
            s.token[i], s.score[i] = self.token[i].data_ptr(), self.score[i].data_ptr()
            s.node[i], s.key[i] = self.node[i].data_ptr(), self.key[i].data_ptr()
        self.parents = torch.zeros((L + 1, R_max), dtype=torch.int32, device=dev)
        self.out_flat = torch.zeros(R_max, dtype=torch.int32, device=dev)
        s.parents, s.out_flat = self.parents.data_ptr(), self.out_flat.data_ptr()
        # activations
        # residual stream: fp32, or bf16 (half the traffic of every LayerNorm and residual projection)
        self.x = torch.zeros((R_max, d_model), dtype=torch.bfloat16 if residual_bf16 else torch.float32, device=dev)
        self.h = torch.zeros((R_max, max(d_model, d_ffn)), dtype=torch.bfloat16, device=dev)
        self.qkv = torch.zeros((R_max, max(3 * HD, d_ffn)), dtype=torch.bfloat16, device=dev)
        self.attn = torch.zeros((R_max, HD), dtype=torch.bfloat16, device=dev)
        self.logp = torch.zeros((R_max, V), dtype=torch.float32, device=dev)
        self.cand = torch.zeros((R_max, V), dtype=torch.float32, device=dev) if separate_cand else self.logp
        # with row_lse set, `logp` keeps the raw logits and the mask kernel normalises them itself
        self.row_lse = torch.zeros(R_max, dtype=torch.float32, device=dev) if fuse_log_softmax else None
        max_n = max(beam_sizes[t] * V for t in range(L))
        ws_bytes = api.grace_beam_topk_workspace_bytes(B, max_n, max(beam_sizes[1:]))
        self.topk_ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
        self.d_status = torch.zeros(1, dtype=torch.int32, device=dev)
        s.x, s.x_bf16 = (None, self.x.data_ptr()) if residual_bf16 else (self.x.data_ptr(), None)
        # the bf16 stream of the large configurations (tens of MB) fits the persisting part of the L2
        if persist_stream_l2 is None:
            persist_stream_l2 = residual_bf16 and self.x.numel() * 2 >= (8 << 20)
        self.persist_stream_l2 = persist_stream_l2
        self._prepared_streams = set()
        s.h, s.qkv, s.attn, s.logp, s.cand = (self.h.data_ptr(), self.qkv.data_ptr(),
                                                   self.attn.data_ptr(), self.logp.data_ptr(), self.cand.data_ptr())
        s.row_lse = None if self.row_lse is None else self.row_lse.data_ptr()
        # Candidates are not materialised unless asked for (or needed: no fused log-softmax, or a separate
        # candidate buffer for inspection): the mask kernel then leaves allow bits, the top-k reads the logits
        # through them.
        if materialize_cand is None:
            materialize_cand = separate_cand or not fuse_log_softmax
        self.allow_bits = None if materialize_cand else torch.zeros((R_max, V // 64), dtype=torch.int64, device=dev)
        s.allow_bits = None if self.allow_bits is None else self.allow_bits.data_ptr()
        # The allow-bits path pays off where few tokens of a row survive the catalog mask.  Children per node are
        # known from the trie: a beam of step t sits on a node of level t and has (nodes of level t+1) / (nodes of
        # level t) children on average; steps whose rows keep more than 2 % of the codebook materialise candidates.
        self.masked_from_step = 0
        if self.allow_bits is not None and level_start is not None:
            sizes = np.diff(np.asarray(level_start, dtype=np.int64))          # nodes per level 0..L
            for t in range(L):
                if sizes[t + 1] / max(1, sizes[t]) / V > 0.02:
                    self.masked_from_step = t + 1
        # log-sum-exp partials from the logits GEMM's epilogue (one pair per row and 256-column tile)
        self.lse_part = (torch.zeros((R_max, V // 256, 2), dtype=torch.float32, device=dev)
                         if (fuse_log_softmax and lse_from_gemm and V % 256 == 0 and V // 256 <= 32) else None)
        s.lse_part = None if self.lse_part is None else self.lse_part.data_ptr()
        # On the allow-bits steps the constraint can run before the logits GEMM, which then stores only the allowed
        # logits: self.logp is valid only where a token is allowed on those steps.
        self.logits_allowed_only = bool(logits_allowed_only and self.allow_bits is not None and self.lse_part is not None
                                        and self.row_lse is not None)
        s.logits_allowed_only = int(self.logits_allowed_only)
        # With the allowed-only logits GEMM the dense trie level costs the same either way (measured: step 1 of the
        # serving-scale loop 3.64 ms both ways), so every step selects through the allow bits and neither the
        # logits nor the candidates are ever written out in full.
        if self.logits_allowed_only:
            self.masked_from_step = 0
        if masked_from_step is not None and self.allow_bits is not None:
            self.masked_from_step = int(masked_from_step)
        s.masked_from_step = self.masked_from_step
        self.row_affine = torch.zeros((R_max, 2), dtype=torch.float32, device=dev) if fold_layer_norm else None
        s.row_affine = None if self.row_affine is None else self.row_affine.data_ptr()
        s.topk_ws, s.topk_ws_bytes, s.d_status = self.topk_ws.data_ptr(), ws_bytes, self.d_status.data_ptr()
        self.struct = s
        code = api.grace_decoder_validate(s)
        if code != api.GRACE_OK:
            raise api.GraceError(code, "grace_decoder_validate")

    # ---- once per request batch: cross-attention K/V from the encoder output (Section 3.2) ----
    def project_cross_kv(self, enc: torch.Tensor) -> None:
        """enc bf16 [B, T_ctx, d_enc] -> k_cross / v_cross [B, T_ctx, H, d_h] per layer."""
        B, T, d_enc = enc.shape
        x = enc.reshape(B * T, d_enc)
        for li in range(self.n_layers):
            api.grace_linear(x, self.w_kc[li], self.k_cross[li].view(B * T, -1))
            api.grace_linear(x, self.w_vc[li], self.v_cross[li].view(B * T, -1))

    def reset(self) -> None:
        """Start state (Section 3.3: M_0 = 1): start token, score 0, root node, empty key."""
        api.grace_decode_begin(self.struct)

    def prepare_stream(self) -> None:
        """Once per CUDA stream the decoder is used on (before any graph capture on it): asks for the residual
        stream to stay resident in L2 (it is re-read nine times per layer while larger tensors stream past)."""
        sid = torch.cuda.current_stream(self.device).cuda_stream
        if self.persist_stream_l2 and sid not in self._prepared_streams:
            try:
                api.grace_stream_l2_persist(self.x)
            except api.GraceError:                         # a residency hint the device refuses is not an error
                self.persist_stream_l2 = False
            self._prepared_streams.add(sid)

    def step(self, t: int) -> None:
        if self.persist_stream_l2 and not torch.cuda.is_current_stream_capturing():
            self.prepare_stream()
        api.grace_decode_step(self.struct, t)

    def decode(self) -> None:
        for t in range(self.L):
            self.step(t)

    def serve(self, enc_hosts, outputs) -> None:
        """Decode a sequence of batches whose encoder outputs sit in PINNED host memory.

        enc_hosts: sequence of pinned bf16 tensors [B, T_ctx, d_enc]; outputs: sequence (same length) of dicts
        with pinned host tensors 'score' fp32 [B*K], 'key' int64 [B*K], 'node' int32 [B*K] that receive the final
        beam of that batch.  Host copies run on a second stream: the input of batch i+1 travels while batch i
        computes (two device buffers), results leave while the next cross-K/V projection runs.  Returns after a
        device-wide synchronize, when every output is complete.
        """
        n = len(enc_hosts)
        if n == 0:
            return
        K, fin = self.beam_sizes[-1], self.L & 1
        rows = self.B * K
        comp = torch.cuda.current_stream()
        copy = torch.cuda.Stream()
        enc_dev = [torch.empty_like(enc_hosts[0], device=self.device) for _ in range(2)]
        ev_in = [torch.cuda.Event() for _ in range(2)]       # input buffer filled
        ev_free = [torch.cuda.Event() for _ in range(2)]     # input buffer consumed by the projection
        ev_done, ev_out = torch.cuda.Event(), torch.cuda.Event()
        for ev in ev_free:
            ev.record(comp)
        ev_out.record(copy)

        def send(i):
            if i >= n:
                return
            with torch.cuda.stream(copy):
                copy.wait_event(ev_free[i & 1])
                enc_dev[i & 1].copy_(enc_hosts[i], non_blocking=True)
                ev_in[i & 1].record(copy)

        send(0)
        for i in range(n):
            comp.wait_event(ev_in[i & 1])
            self.project_cross_kv(enc_dev[i & 1])
            ev_free[i & 1].record(comp)
            send(i + 1)                                       # the next input travels under this batch's compute
            comp.wait_event(ev_out)                           # the previous results have left the state buffers
            self.reset()
            self.decode()
            ev_done.record(comp)
            with torch.cuda.stream(copy):
                copy.wait_event(ev_done)
                outputs[i]["score"].copy_(self.score[fin][:rows], non_blocking=True)
                outputs[i]["key"].copy_(self.key[fin][:rows], non_blocking=True)
                outputs[i]["node"].copy_(self.node[fin][:rows], non_blocking=True)
                ev_out.record(copy)
        torch.cuda.synchronize()

    def log_probs(self, rows: int) -> torch.Tensor:
        """Log-probabilities of the last step's first `rows` rows (reconstructed from logits and the row
        log-sum-exp when the log-softmax is fused into the mask kernel; needs separate_cand)."""
        if self.row_lse is None:
            return self.logp[:rows]
        return self.logp[:rows] - self.row_lse[:rows, None]

    def results(self):
        """(sids int64 [B, K, L], score [B, K], node [B, K]) read back by following the parents."""
        L, B, K = self.L, self.B, self.beam_sizes[-1]
        fin = L & 1
        score = self.score[fin][: B * K].view(B, K).cpu().numpy()
        node = self.node[fin][: B * K].view(B, K).cpu().numpy()
        key = self.key[fin][: B * K].view(B, K).cpu().numpy().view(np.uint64)
        sids = np.zeros((B, K, L), dtype=np.int64)
        for j in range(L):
            sids[:, :, j] = ((key >> np.uint64(16 * j)) & np.uint64(0xFFFF)).astype(np.int64) - 1
        return sids, score, node
