// One decode step of the GTM-constrained beam search (Sections 3.1-3.3): decoder layers on the
// current beam rows, log-probabilities, CD + GTM mask with score add, beam top-k, state update.
// Host-side sequencing only; every stage is one of the library's own kernels on the caller's
// stream, with no allocation and no synchronisation, so the loop can be enqueued back to back.
#include "common.cuh"

extern "C" grace_status_t grace_decoder_validate(const grace_decoder_t* d) {
  if (!d) return GRACE_INVALID_ARG;
  if (d->B <= 0 || d->n_layers <= 0 || d->n_layers > GRACE_MAX_LAYERS || d->L <= 0 || d->L > 4 ||
      d->L > GRACE_MAX_STEPS || d->H <= 0 || d->T_ctx <= 0)
    return GRACE_INVALID_ARG;
  if ((d->d_h != 32 && d->d_h != 64 && d->d_h != 128) || d->d_model % 64 || d->d_ffn % 64 ||
      (d->H * d->d_h) % 64 || d->V % 64 || d->V <= 0 || d->V >= 65535 || d->d_model > (d->x ? 4096 : 2048) || d->H * d->d_h > 8192)
    return GRACE_UNSUPPORTED_SHAPE;
  int64_t mmax = 0;
  for (int t = 0; t <= d->L; ++t) {
    if (d->beam_sizes[t] <= 0) return GRACE_INVALID_ARG;
    if (t < d->L && d->beam_sizes[t] > mmax) mmax = d->beam_sizes[t];
    if (d->beam_sizes[t] > 4096) return GRACE_UNSUPPORTED_SHAPE;
  }
  if (d->beam_sizes[d->L] > mmax) mmax = d->beam_sizes[d->L];
  if (d->R_max < (int64_t)d->B * mmax) return GRACE_INVALID_ARG;
  for (int l = 0; l < d->n_layers; ++l) {
    const grace_layer_t& w = d->layers[l];
    if (!w.ln1_g || !w.ln1_b || !w.ln2_g || !w.ln2_b || !w.ln3_g || !w.ln3_b || !w.w_qkv || !w.w_o || !w.w_qc ||
        !w.w_oc || !w.w_1 || !w.w_2 || !w.k_cross || !w.v_cross || (!w.qkv_slabs && (!w.k_cache || !w.v_cache)))
      return GRACE_INVALID_ARG;
  }
  if (!d->embed || !d->pos || !d->lnf_g || !d->lnf_b || !d->w_out || !d->parents || (!d->x && !d->x_bf16) || !d->h || !d->qkv ||
      !d->attn || !d->logp || !d->cand || !d->topk_ws || !d->out_flat)
    return GRACE_INVALID_ARG;
  if (d->row_affine != nullptr) {                          // folded LayerNorms: bf16 stream and every bias vector
    if (!d->x_bf16 || d->x || !d->cb_out) return GRACE_INVALID_ARG;        // (column sums: none = centred stream)
    for (int l = 0; l < d->n_layers; ++l) {
      const grace_layer_t& w = d->layers[l];
      if (!w.cb_qkv || !w.cb_qc || !w.cb_1) return GRACE_INVALID_ARG;
    }
  }
  if (d->logits_allowed_only && (!d->allow_bits || !d->row_lse || !d->lse_part)) return GRACE_INVALID_ARG;
  for (int i = 0; i < 2; ++i)
    if (!d->token[i] || !d->score[i] || !d->node[i] || !d->key[i]) return GRACE_INVALID_ARG;
  if (d->trie.V != d->V || d->trie.L != d->L || !d->trie.child_bits || !d->trie.child_base) return GRACE_INVALID_ARG;
  return GRACE_OK;
}

namespace grace {
__global__ void decode_begin_kernel(int32_t* token, float* score, int32_t* node, uint64_t* key, int32_t* d_status,
                                    int rows, int start_token) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < rows) { token[i] = start_token; score[i] = 0.f; node[i] = 0; key[i] = 0ull; }
  if (i == 0 && d_status != nullptr) *d_status = 0;
}
}  // namespace grace

extern "C" grace_status_t grace_decode_begin(const grace_decoder_t* d, void* stream) {
  grace_status_t st = grace_decoder_validate(d);
  if (st != GRACE_OK) return st;
  const int rows = d->B * d->beam_sizes[0];
  grace::decode_begin_kernel<<<(rows + 255) / 256, 256, 0, (cudaStream_t)stream>>>(
      d->token[0], d->score[0], d->node[0], d->key[0], d->d_status, rows, d->V);
  GRACE_LAUNCH_CHECK();
  return GRACE_OK;
}

#define GRACE_TRY(expr)                         \
  do {                                          \
    grace_status_t _s = (expr);                 \
    if (_s != GRACE_OK) return _s;              \
  } while (0)

extern "C" grace_status_t grace_decode_step(const grace_decoder_t* d, int t, void* stream) {
  GRACE_TRY(grace_decoder_validate(d));
  if (t < 0 || t >= d->L) return GRACE_INVALID_ARG;
  const int cur = t & 1, nxt = cur ^ 1;
  const int B = d->B, M = d->beam_sizes[t], K = d->beam_sizes[t + 1];
  const int R = B * M;
  const int D = d->d_model, HD = d->H * d->d_h;
  const float scale = 1.0f / sqrtf((float)d->d_h);
  int32_t* st = d->d_status;

  // residual stream: fp32 (x) or bf16 (x_bf16)
  const bool xb = (d->x == nullptr);
  auto layer_norm = [&](const float* g, const float* b) -> grace_status_t {
    return xb ? grace_layer_norm_bf16(d->x_bf16, g, b, d->h, R, D, d->ln_eps, stream)
              : grace_layer_norm(d->x, g, b, d->h, R, D, d->ln_eps, stream);
  };
  // LayerNorm + the GEMM that consumes it: either the two kernels, or (folded) row statistics + a GEMM on the
  // raw stream whose epilogue applies them
  const bool folded = xb && d->row_affine != nullptr;
  auto ln_linear = [&](const float* g, const float* b, const uint16_t* w, const float* cs, const float* cb,
                       uint16_t* y_bf16, float* y_f32, int64_t ldy, int N, int relu, float* lse_part) -> grace_status_t {
    if (folded)
      return grace_linear_layer_norm(d->x_bf16, D, w, D, d->ln_eps, d->row_affine, cs, cb, y_bf16, y_f32, ldy, lse_part, R,
                                     N, D, relu, stream);
    grace_status_t s1 = layer_norm(g, b);
    if (s1 != GRACE_OK) return s1;
    if (lse_part != nullptr) return grace_linear_f32_lse(d->h, D, w, D, y_f32, ldy, lse_part, R, N, D, stream);
    return grace_linear(d->h, D, w, D, y_bf16, y_f32, ldy, nullptr, R, N, D, relu, stream);
  };
  auto add_into_x = [&](const uint16_t* a, int64_t lda, const uint16_t* w, int K) -> grace_status_t {
    return xb ? grace_linear_add_bf16(a, lda, w, K, d->x_bf16, D, R, D, K, stream)
              : grace_linear(a, lda, w, K, nullptr, d->x, D, d->x, R, D, K, 0, stream);
  };
  if (xb) GRACE_TRY(grace_embed_bf16(d->token[cur], d->embed, d->pos + (int64_t)t * D, d->x_bf16, R, D, d->V + 1, st, stream));
  else GRACE_TRY(grace_embed(d->token[cur], d->embed, d->pos + (int64_t)t * D, d->x, R, D, d->V + 1, st, stream));
  for (int l = 0; l < d->n_layers; ++l) {
    const grace_layer_t& w = d->layers[l];
    // self-attention block
    if (w.qkv_slabs != nullptr) {                          // the projection lands in the cache slab of this step
      const int64_t slab = d->R_max * 3 * (int64_t)HD;
      GRACE_TRY(ln_linear(w.ln1_g, w.ln1_b, w.w_qkv, w.cs_qkv, w.cb_qkv, w.qkv_slabs + t * slab, nullptr, 3 * HD, 3 * HD,
                          0, nullptr));
      GRACE_TRY(grace_self_attn_inplace(w.qkv_slabs, 3 * HD, slab, d->parents, d->beam_sizes, d->attn, HD, B, t,
                                        d->H, d->d_h, d->R_max, scale, st, stream));
    } else {
      GRACE_TRY(ln_linear(w.ln1_g, w.ln1_b, w.w_qkv, w.cs_qkv, w.cb_qkv, d->qkv, nullptr, 3 * HD, 3 * HD, 0, nullptr));
      GRACE_TRY(grace_self_attn(d->qkv, 3 * HD, w.k_cache, w.v_cache, d->parents, d->beam_sizes, d->attn, HD,
                                B, t, d->H, d->d_h, d->R_max, scale, st, stream));
    }
    GRACE_TRY(add_into_x(d->attn, HD, w.w_o, HD));
    // cross-attention block
    GRACE_TRY(ln_linear(w.ln2_g, w.ln2_b, w.w_qc, w.cs_qc, w.cb_qc, d->qkv, nullptr, HD, HD, 0, nullptr));
    GRACE_TRY(grace_cross_attn(d->qkv, HD, w.k_cross, w.v_cross, (int64_t)d->T_ctx * HD, d->d_h, HD, d->attn, HD,
                               nullptr, B, M, d->H, d->d_h, d->T_ctx, scale, st, stream));
    GRACE_TRY(add_into_x(d->attn, HD, w.w_oc, HD));
    // feed-forward block
    GRACE_TRY(ln_linear(w.ln3_g, w.ln3_b, w.w_1, w.cs_1, w.cb_1, d->qkv, nullptr, d->d_ffn, d->d_ffn, 1, nullptr));
    GRACE_TRY(add_into_x(d->qkv, d->d_ffn, w.w_2, d->d_ffn));
  }
  // the logits GEMM can leave the rows' log-sum-exp partials (large steps), the mask kernel then merges them
  const int n_parts = d->V / 256;
  const bool parts = d->lse_part != nullptr && d->row_lse != nullptr && R >= 1024 && (d->V % 256) == 0 && n_parts <= 32;
  int32_t* parent_out = d->parents + (int64_t)(t + 1) * d->R_max;
  if (parts && d->logits_allowed_only && d->allow_bits != nullptr && t >= d->masked_from_step) {
    // The constraint first (it needs the beam state only), then a logits GEMM that stores only the allowed logits
    // and the rows' log-sum-exp partials, their merge, and the selection through the allow bits: neither the
    // logits tensor nor the candidates are written out.
    GRACE_TRY(grace_gtm_allow_bits(d->node[cur], d->key[cur], &d->trie, &d->matcher, d->allow_bits, B, M, d->V, t, st,
                                   stream));
    if (folded)
      GRACE_TRY(grace_linear_logits_allowed(d->x_bf16, D, d->w_out, D, d->ln_eps, d->row_affine, d->cs_out, d->cb_out,
                                            d->allow_bits, d->logp, d->V, d->lse_part, R, d->V, D, stream));
    else {
      GRACE_TRY(layer_norm(d->lnf_g, d->lnf_b));
      GRACE_TRY(grace_linear_logits_allowed(d->h, D, d->w_out, D, 0.f, nullptr, nullptr, nullptr, d->allow_bits, d->logp,
                                            d->V, d->lse_part, R, d->V, D, stream));
    }
    GRACE_TRY(grace_row_lse_from_parts(d->lse_part, n_parts, d->node[cur], &d->trie, d->row_lse, R, stream));
    GRACE_TRY(grace_beam_topk_masked(d->logp, d->allow_bits, d->score[cur], d->row_lse, B, M, d->V, K, d->score[nxt],
                                     d->out_flat, parent_out, d->token[nxt], d->topk_ws, d->topk_ws_bytes, st, stream));
    GRACE_TRY(grace_beam_update(parent_out, d->token[nxt], d->score[nxt], d->node[cur], d->key[cur], &d->trie,
                                d->node[nxt], d->key[nxt], B, K, M, t, st, stream));
    return GRACE_OK;
  }
  GRACE_TRY(ln_linear(d->lnf_g, d->lnf_b, d->w_out, d->cs_out, d->cb_out, nullptr, d->logp, d->V, d->V, 0,
                      parts ? d->lse_part : nullptr));
  // log-softmax, CD + GTM mask and score add: one fused kernel when row_lse is provided
  if (d->row_lse != nullptr && d->allow_bits != nullptr && t >= d->masked_from_step) {
    // candidates never materialised: the mask kernel leaves the allow bits and the rows' log-sum-exp, the
    // selection reads the logits through them (and only where a token is allowed)
    GRACE_TRY(grace_gtm_mask_logits_parts(d->logp, d->row_lse, d->score[cur], d->node[cur], d->key[cur], &d->trie,
                                          &d->matcher, nullptr, d->allow_bits, B, M, d->V, t,
                                          parts ? d->lse_part : nullptr, n_parts, st, stream));
    GRACE_TRY(grace_beam_topk_masked(d->logp, d->allow_bits, d->score[cur], d->row_lse, B, M, d->V, K, d->score[nxt],
                                     d->out_flat, parent_out, d->token[nxt], d->topk_ws, d->topk_ws_bytes, st, stream));
    GRACE_TRY(grace_beam_update(parent_out, d->token[nxt], d->score[nxt], d->node[cur], d->key[cur], &d->trie,
                                d->node[nxt], d->key[nxt], B, K, M, t, st, stream));
    return GRACE_OK;
  }
  if (d->row_lse != nullptr) {
    GRACE_TRY(grace_gtm_mask_logits_parts(d->logp, d->row_lse, d->score[cur], d->node[cur], d->key[cur], &d->trie,
                                          &d->matcher, d->cand, nullptr, B, M, d->V, t,
                                          parts ? d->lse_part : nullptr, n_parts, st, stream));
  } else {
    GRACE_TRY(grace_log_softmax(d->logp, R, d->V, stream));
    GRACE_TRY(grace_gtm_mask(d->logp, d->score[cur], d->node[cur], d->key[cur], &d->trie, &d->matcher, d->cand,
                             nullptr, B, M, d->V, t, st, stream));
  }
  // parents of step t+1 live in slab t+1; tokens become the next step's input tokens
  GRACE_TRY(grace_beam_topk(d->cand, B, (int64_t)M * d->V, K, d->V, d->score[nxt], d->out_flat, parent_out,
                            d->token[nxt], d->topk_ws, d->topk_ws_bytes, st, stream));
  GRACE_TRY(grace_beam_update(parent_out, d->token[nxt], d->score[nxt], d->node[cur], d->key[cur], &d->trie,
                              d->node[nxt], d->key[nxt], B, K, M, t, st, stream));
  return GRACE_OK;
}

namespace grace {
int linear_tc_timeouts();
int cross_attn_tc_timeouts();
}  // namespace grace

extern "C" int grace_wait_timeouts(void) {
  const int a = grace::linear_tc_timeouts(), b = grace::cross_attn_tc_timeouts();
  return (a < 0 || b < 0) ? -1 : a + b;
}

// Keeps part of a buffer that many kernels of a step re-read (the residual stream: three add-reductions,
// three statistics passes and three GEMM operand reads per layer) resident in L2 across the large tensors
// that stream past it: an access-policy window on the stream, backed by this context's persisting carve-out.
// A refused hint must not leave a stale "last error" behind for the next launch check to find.
#define L2_TRY(expr)                                          \
  do {                                                        \
    if ((expr) != cudaSuccess) {                              \
      (void)cudaGetLastError();                               \
      return GRACE_CUDA_ERROR;                                \
    }                                                         \
  } while (0)
extern "C" grace_status_t grace_stream_l2_persist(void* stream, const void* ptr, size_t bytes, float fraction) {
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaStreamAttrValue v;
  memset(&v, 0, sizeof(v));
  if (ptr == nullptr || bytes == 0) {                       // clear the window
    v.accessPolicyWindow.hitProp = cudaAccessPropertyNormal;
    v.accessPolicyWindow.missProp = cudaAccessPropertyNormal;
    L2_TRY(cudaStreamSetAttribute(s, cudaStreamAttributeAccessPolicyWindow, &v));
    return GRACE_OK;
  }
  if (!(fraction > 0.f && fraction <= 1.f)) return GRACE_INVALID_ARG;
  int dev = 0, max_persist = 0, max_window = 0;
  L2_TRY(cudaGetDevice(&dev));
  L2_TRY(cudaDeviceGetAttribute(&max_persist, cudaDevAttrMaxPersistingL2CacheSize, dev));
  L2_TRY(cudaDeviceGetAttribute(&max_window, cudaDevAttrMaxAccessPolicyWindowSize, dev));
  if (max_persist <= 0 || max_window <= 0) return GRACE_UNSUPPORTED_SHAPE;
  const size_t window = bytes < (size_t)max_window ? bytes : (size_t)max_window;
  size_t carve = (size_t)((double)window * fraction);
  if (carve > (size_t)max_persist) carve = (size_t)max_persist;
  L2_TRY(cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, carve));
  v.accessPolicyWindow.base_ptr = const_cast<void*>(ptr);
  v.accessPolicyWindow.num_bytes = window;
  v.accessPolicyWindow.hitRatio = (float)((double)carve / (double)window);   // the share of the window's lines kept
  v.accessPolicyWindow.hitProp = cudaAccessPropertyPersisting;
  v.accessPolicyWindow.missProp = cudaAccessPropertyNormal;
  L2_TRY(cudaStreamSetAttribute(s, cudaStreamAttributeAccessPolicyWindow, &v));
  return GRACE_OK;
}
#undef L2_TRY
