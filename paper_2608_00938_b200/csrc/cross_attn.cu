// Cross-attention in the beam-as-query layout (Section 5.1, Appendix B): the M beams of a request
// are M query rows against that request's one copy of K and V.
//
// Four kernels behind one entry point:
//   * cross_attn_ms_kernel (cross_attn_ms.cuh): tcgen05 / TMEM / TMA, four softmax streams per SM,
//     head size 64: the serving shapes.
//   * cross_attn_tc_kernel (cross_attn_tc.cuh): tcgen05 / TMEM / TMA flash attention, head size 128.
//   * cross_attn_row_kernel (below): a handful of query rows per request (step 0 of a decode).
//   * cross_attn_small_kernel (below): a plain CUDA-core kernel for everything else (tiny
//     configurations, d_h = 32, per-request encoder lengths at head size 128).  One warp per (row,
//     head); lanes split the encoder positions for the scores and the head dimension for the sum.
#include "common.cuh"
#include "cross_attn_tc.cuh"
#include "cross_attn_ms.cuh"


namespace grace {

struct CrossSmallParams {
  const uint16_t* q; const uint16_t* k; const uint16_t* v; uint16_t* out; float* lse;
  int64_t q_row_stride, out_row_stride, kv_stride_b, kv_stride_h, kv_stride_t;
  int R, M, H, T_ctx; float scale;
  const int32_t* enc_len;        // nullable: valid encoder positions per request (small kernel only)
};

template <int DH>
__global__ void __launch_bounds__(128)
cross_attn_small_kernel(const CrossSmallParams p) {
  constexpr int kChunk = 128;                 // encoder positions per round
  constexpr int kPerLane = DH / 32;           // output elements per lane
  __shared__ float probs[4][kChunk];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t item = (int64_t)blockIdx.x * 4 + warp;      // (row, head)
  if (item >= (int64_t)p.R * p.H) return;
  const int r = (int)(item / p.H), h = (int)(item % p.H);
  const int b = r / p.M;
  int T = p.T_ctx;                             // valid encoder positions of this request
  if (p.enc_len != nullptr) { const int e = __ldg(p.enc_len + b); T = e < 0 ? 0 : (e < T ? e : T); }
  const uint16_t* qp = p.q + (int64_t)r * p.q_row_stride + h * DH;
  const uint16_t* kb = p.k + (int64_t)b * p.kv_stride_b + (int64_t)h * p.kv_stride_h;
  const uint16_t* vb = p.v + (int64_t)b * p.kv_stride_b + (int64_t)h * p.kv_stride_h;
  uint32_t qreg[DH / 2];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) {
    const uint4 t4 = __ldg(reinterpret_cast<const uint4*>(qp) + i);
    qreg[4 * i] = t4.x; qreg[4 * i + 1] = t4.y; qreg[4 * i + 2] = t4.z; qreg[4 * i + 3] = t4.w;
  }
  float m_run = -INFINITY, l_run = 0.f;
  float acc[kPerLane];
#pragma unroll
  for (int j = 0; j < kPerLane; ++j) acc[j] = 0.f;
  for (int t0 = 0; t0 < T; t0 += kChunk) {
    float s[kChunk / 32];
    float cmax = -INFINITY;
#pragma unroll
    for (int i = 0; i < kChunk / 32; ++i) {
      const int t = t0 + i * 32 + lane;
      s[i] = -INFINITY;
      if (t < T) {
        const uint4* kr = reinterpret_cast<const uint4*>(kb + (int64_t)t * p.kv_stride_t);
        float d = 0.f;
#pragma unroll
        for (int c = 0; c < DH / 8; ++c) {
          const uint4 kk = __ldg(kr + c);
          d = fmaf(bf16_lo(qreg[4 * c]), bf16_lo(kk.x), d);     d = fmaf(bf16_hi(qreg[4 * c]), bf16_hi(kk.x), d);
          d = fmaf(bf16_lo(qreg[4 * c + 1]), bf16_lo(kk.y), d); d = fmaf(bf16_hi(qreg[4 * c + 1]), bf16_hi(kk.y), d);
          d = fmaf(bf16_lo(qreg[4 * c + 2]), bf16_lo(kk.z), d); d = fmaf(bf16_hi(qreg[4 * c + 2]), bf16_hi(kk.z), d);
          d = fmaf(bf16_lo(qreg[4 * c + 3]), bf16_lo(kk.w), d); d = fmaf(bf16_hi(qreg[4 * c + 3]), bf16_hi(kk.w), d);
        }
        s[i] = d * p.scale;
      }
      cmax = fmaxf(cmax, s[i]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cmax = fmaxf(cmax, __shfl_xor_sync(kFullMask, cmax, o));
    const float m_new = fmaxf(m_run, cmax);
    const float corr = __expf(m_run - m_new);            // 0 on the first round (m_run = -inf)
    float csum = 0.f;
    __syncwarp();
#pragma unroll
    for (int i = 0; i < kChunk / 32; ++i) {
      const float e = (t0 + i * 32 + lane < T) ? __expf(s[i] - m_new) : 0.f;
      probs[warp][i * 32 + lane] = e;
      csum += e;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) csum += __shfl_xor_sync(kFullMask, csum, o);
    l_run = l_run * corr + csum;
    m_run = m_new;
    __syncwarp();
#pragma unroll
    for (int j = 0; j < kPerLane; ++j) acc[j] *= corr;
    const int tn = min(kChunk, T - t0);
    for (int tt = 0; tt < tn; ++tt) {
      const float w = probs[warp][tt];
      const uint16_t* vr = vb + (int64_t)(t0 + tt) * p.kv_stride_t;
#pragma unroll
      for (int j = 0; j < kPerLane; ++j)
        acc[j] = fmaf(w, __uint_as_float((uint32_t)__ldg(vr + j * 32 + lane) << 16), acc[j]);
    }
  }
  const float inv = l_run > 0.f ? 1.f / l_run : 0.f;          // no encoder position: the output is defined as zero
  uint16_t* op = p.out + (int64_t)r * p.out_row_stride + h * DH;
#pragma unroll
  for (int j = 0; j < kPerLane; ++j) {
    __nv_bfloat16 o = __float2bfloat16_rn(acc[j] * inv);
    op[j * 32 + lane] = *reinterpret_cast<uint16_t*>(&o);
  }
  if (p.lse != nullptr && lane == 0) p.lse[(int64_t)r * p.H + h] = l_run > 0.f ? m_run + logf(l_run) : -INFINITY;
}

// A handful of query rows per request (step 0 of a decode: one beam per request): the tensor-core kernel would
// run one 128-row tile with a single live row through all K/V blocks in sequence.  Here a CTA owns one
// (row, head) and its eight warps split the encoder positions; inside a warp DH/8 lanes share a position
// (16 bytes of the K / V row each, so a row is one coalesced run), every lane group keeps an online-softmax
// state (running maximum, sum, DH/G-element slice of the weighted sum), and the 8 x 32/G states are merged
// through shared memory at the end.  All arithmetic in fp32.
template <int DH>
__global__ void __launch_bounds__(256)
cross_attn_row_kernel(const CrossSmallParams p) {
  pdl_wait();
  pdl_trigger();
  constexpr int G = DH / 8;                   // lanes per encoder position
  constexpr int RP = 32 / G;                  // positions per warp pass
  constexpr int kWarps = 8, kStates = kWarps * RP;
  __shared__ float st_m[kStates], st_l[kStates], st_acc[kStates][DH];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int piece = lane % G, grp = lane / G;
  const int r = blockIdx.x / p.H, h = blockIdx.x % p.H;
  const int b = r / p.M;
  const uint16_t* kb = p.k + (int64_t)b * p.kv_stride_b + (int64_t)h * p.kv_stride_h + piece * 8;
  const uint16_t* vb = p.v + (int64_t)b * p.kv_stride_b + (int64_t)h * p.kv_stride_h + piece * 8;
  float q[8];
  {
    const uint4 t4 = __ldg(reinterpret_cast<const uint4*>(p.q + (int64_t)r * p.q_row_stride + h * DH) + piece);
    q[0] = bf16_lo(t4.x) * p.scale; q[1] = bf16_hi(t4.x) * p.scale; q[2] = bf16_lo(t4.y) * p.scale; q[3] = bf16_hi(t4.y) * p.scale;
    q[4] = bf16_lo(t4.z) * p.scale; q[5] = bf16_hi(t4.z) * p.scale; q[6] = bf16_lo(t4.w) * p.scale; q[7] = bf16_hi(t4.w) * p.scale;
  }
  // this warp's contiguous slice of the encoder positions, RP at a time
  const int per_warp = (p.T_ctx + kWarps - 1) / kWarps;
  const int t_begin = warp * per_warp, t_end = min(p.T_ctx, t_begin + per_warp);
  float m_run = -INFINITY, l_run = 0.f;
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  // The op is bound by reading K and V once (a row per request: nothing is reused), so loads never stop: the
  // pieces of the next four passes are requested before the current four are used.
  constexpr int U = 4;
  uint4 kk[U], vv[U], kn[U], vn[U];
  auto fetch = [&](int t0, uint4 (&kd)[U], uint4 (&vd)[U]) {
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int t = t0 + u * RP + grp;
      const int64_t off = (int64_t)(t < t_end ? t : t_begin) * p.kv_stride_t;
      kd[u] = __ldg(reinterpret_cast<const uint4*>(kb + off));
      vd[u] = __ldg(reinterpret_cast<const uint4*>(vb + off));
    }
  };
  if (t_begin < t_end) fetch(t_begin, kk, vv);
  for (int t0 = t_begin; t0 < t_end; t0 += U * RP) {
    if (t0 + U * RP < t_end) fetch(t0 + U * RP, kn, vn);
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const bool live = t0 + u * RP + grp < t_end;
      float d = q[0] * bf16_lo(kk[u].x);
      d = fmaf(q[1], bf16_hi(kk[u].x), d); d = fmaf(q[2], bf16_lo(kk[u].y), d); d = fmaf(q[3], bf16_hi(kk[u].y), d);
      d = fmaf(q[4], bf16_lo(kk[u].z), d); d = fmaf(q[5], bf16_hi(kk[u].z), d); d = fmaf(q[6], bf16_lo(kk[u].w), d);
      d = fmaf(q[7], bf16_hi(kk[u].w), d);
#pragma unroll
      for (int o = 1; o < G; o <<= 1) d += __shfl_xor_sync(kFullMask, d, o);
      if (live) {
        const float m_new = fmaxf(m_run, d);
        const float corr = __expf(m_run - m_new);          // 0 the first time (m_run = -inf)
        const float w = __expf(d - m_new);
        l_run = fmaf(l_run, corr, w);
        acc[0] = fmaf(acc[0], corr, w * bf16_lo(vv[u].x)); acc[1] = fmaf(acc[1], corr, w * bf16_hi(vv[u].x));
        acc[2] = fmaf(acc[2], corr, w * bf16_lo(vv[u].y)); acc[3] = fmaf(acc[3], corr, w * bf16_hi(vv[u].y));
        acc[4] = fmaf(acc[4], corr, w * bf16_lo(vv[u].z)); acc[5] = fmaf(acc[5], corr, w * bf16_hi(vv[u].z));
        acc[6] = fmaf(acc[6], corr, w * bf16_lo(vv[u].w)); acc[7] = fmaf(acc[7], corr, w * bf16_hi(vv[u].w));
        m_run = m_new;
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) { kk[u] = kn[u]; vv[u] = vn[u]; }
  }
  const int state = warp * RP + grp;
  if (piece == 0) { st_m[state] = m_run; st_l[state] = l_run; }
#pragma unroll
  for (int i = 0; i < 8; ++i) st_acc[state][piece * 8 + i] = acc[i];
  __syncthreads();
  if (threadIdx.x < DH) {
    float m_all = -INFINITY;
    for (int s2 = 0; s2 < kStates; ++s2) m_all = fmaxf(m_all, st_m[s2]);
    float l_all = 0.f, o = 0.f;
    for (int s2 = 0; s2 < kStates; ++s2) {
      const float f = st_m[s2] == -INFINITY ? 0.f : __expf(st_m[s2] - m_all);   // a state that saw no position
      l_all = fmaf(st_l[s2], f, l_all);
      o = fmaf(st_acc[s2][threadIdx.x], f, o);
    }
    __nv_bfloat16 ob = __float2bfloat16_rn(o / l_all);
    p.out[(int64_t)r * p.out_row_stride + h * DH + threadIdx.x] = *reinterpret_cast<uint16_t*>(&ob);
    if (p.lse != nullptr && threadIdx.x == 0) p.lse[(int64_t)r * p.H + h] = m_all + logf(l_all);
  }
}

}  // namespace grace

namespace grace {
int cross_attn_tc_timeouts() { return tc::tc_timeouts_read_and_clear(); }
}  // namespace grace

extern "C" grace_status_t grace_cross_attn_varlen(const uint16_t* q, int64_t q_row_stride,
                                                  const uint16_t* k, const uint16_t* v,
                                                  int64_t kv_stride_b, int64_t kv_stride_h, int64_t kv_stride_t,
                                                  uint16_t* out, int64_t out_row_stride, float* lse,
                                                  const int32_t* enc_len,
                                                  int B, int M, int H, int d_h, int T_ctx, float scale,
                                                  int32_t* d_status, void* stream) {
  using namespace grace;
  (void)d_status;
  if (!q || !k || !v || !out) return GRACE_INVALID_ARG;
  if (B <= 0 || M <= 0 || H <= 0 || T_ctx <= 0 || (int64_t)B * M > 0x7fffffff) return GRACE_INVALID_ARG;
  if (d_h != 32 && d_h != 64 && d_h != 128) return GRACE_UNSUPPORTED_SHAPE;
  if (!grace_aligned16(q) || !grace_aligned16(k) || !grace_aligned16(v) || !grace_aligned16(out) ||
      (q_row_stride & 7) || (out_row_stride & 7) || (kv_stride_b & 7) || (kv_stride_h & 7) || (kv_stride_t & 7) ||
      q_row_stride < (int64_t)H * d_h || out_row_stride < (int64_t)H * d_h || kv_stride_t < d_h)
    return GRACE_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  CrossSmallParams p;
  p.q = q; p.k = k; p.v = v; p.out = out; p.lse = lse;
  p.q_row_stride = q_row_stride; p.out_row_stride = out_row_stride;
  p.kv_stride_b = kv_stride_b; p.kv_stride_h = kv_stride_h; p.kv_stride_t = kv_stride_t;
  p.R = B * M; p.M = M; p.H = H; p.T_ctx = T_ctx; p.scale = scale; p.enc_len = enc_len;
  if (enc_len == nullptr && (d_h == 64 || d_h == 128) && M <= 8 && (int64_t)B * M * H <= 1184) {
    // a few rows per request (step 0 of a decode): one CTA per (row, head), all resident at once
    if (d_h == 64) launch_pdl(cross_attn_row_kernel<64>, dim3(B * M * H), dim3(256), 0, s, p);
    else launch_pdl(cross_attn_row_kernel<128>, dim3(B * M * H), dim3(256), 0, s, p);
    GRACE_LAUNCH_CHECK();
    return GRACE_OK;
  }
  if (cross_attn_ms_supported(B, M, H, d_h, T_ctx) && (enc_len == nullptr || M > 8)) {
    return launch_cross_attn_ms(q, q_row_stride, k, v, kv_stride_b, kv_stride_h, kv_stride_t, out,
                                out_row_stride, lse, enc_len, B, M, H, T_ctx, scale, s);
  }
  if (enc_len == nullptr && cross_attn_tc_supported(B, M, H, d_h, T_ctx)) {
    return launch_cross_attn_tc(q, q_row_stride, k, v, kv_stride_b, kv_stride_h, kv_stride_t, out,
                                out_row_stride, lse, B, M, H, d_h, T_ctx, scale, s);
  }
  const int64_t items = (int64_t)p.R * H;
  const unsigned blocks = (unsigned)((items + 3) / 4);
  switch (d_h) {
    case 32: cross_attn_small_kernel<32><<<blocks, 128, 0, s>>>(p); break;
    case 64: cross_attn_small_kernel<64><<<blocks, 128, 0, s>>>(p); break;
    default: cross_attn_small_kernel<128><<<blocks, 128, 0, s>>>(p); break;
  }
  GRACE_LAUNCH_CHECK();
  return GRACE_OK;
}

extern "C" grace_status_t grace_cross_attn(const uint16_t* q, int64_t q_row_stride,
                                           const uint16_t* k, const uint16_t* v,
                                           int64_t kv_stride_b, int64_t kv_stride_h, int64_t kv_stride_t,
                                           uint16_t* out, int64_t out_row_stride, float* lse,
                                           int B, int M, int H, int d_h, int T_ctx, float scale,
                                           int32_t* d_status, void* stream) {
  return grace_cross_attn_varlen(q, q_row_stride, k, v, kv_stride_b, kv_stride_h, kv_stride_t, out, out_row_stride, lse,
                                 nullptr, B, M, H, d_h, T_ctx, scale, d_status, stream);
}
