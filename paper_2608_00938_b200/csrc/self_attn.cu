// Short-sequence self-attention over a parent-addressed KV cache, fused with the cache write
// (Sections 5.2, 5.3).
//
// The work is HBM-bound: per row a few KB are read and written and almost nothing is computed,
// so no tensor cores and no padded tiles.  One warp owns one beam row.  A row of H * d_h bf16 is
// cut into 16-byte pieces; lane l takes pieces l, l + 32, ...  so every warp access is a run of
// contiguous 512-byte lines.  The warp first resolves the row's ancestor chain (t dependent
// 4-byte loads, warp-uniform, served by L2), then issues all K and V loads of the prefix at
// once, and only then does the arithmetic: dot products reduced over the d_h / 8 lanes of a
// head, fp32 softmax over the <= 8 positions, weighted sum of V.  Beam reordering never moves
// KV: the parent arrays are the block table.  Rows wider than 1024 elements (e.g. 16 heads of 128)
// are cut into 1024-element segments, one warp each (blockIdx.y): heads never interact.
//
// In-place form (grace_self_attn_inplace): the cache slabs ARE the steps' QKV projections ([R_max][3][H][d_h]
// per step, kept), so the K and V of the current token are already where the later steps will look for
// them and the kernel writes nothing but its output: a third less traffic per row at T_self = 2.
#include "common.cuh"

namespace grace {

constexpr int kMaxSelfSteps = 8;            // T_self = t + 1 <= 8

struct SelfAttnParams {
  const uint16_t* qkv;
  uint16_t* k_cache;
  uint16_t* v_cache;
  const int32_t* parents;
  uint16_t* out;
  int32_t* d_status;
  int64_t qkv_row_stride, out_row_stride, R_max;
  int64_t cache_row_stride, cache_slab_stride;   // elements between rows / slabs of k_cache and v_cache
  int write_cache;                               // 0: slab t already holds this step's K and V
  int beam[kMaxSelfSteps];                  // M_0 .. M_t
  int R, t, HD;                             // HD = H * d_h
  float scale;
};

__device__ __forceinline__ float dot8(const uint4& a, const uint4& b) {
  float s = bf16_lo(a.x) * bf16_lo(b.x);
  s = fmaf(bf16_hi(a.x), bf16_hi(b.x), s);
  s = fmaf(bf16_lo(a.y), bf16_lo(b.y), s);
  s = fmaf(bf16_hi(a.y), bf16_hi(b.y), s);
  s = fmaf(bf16_lo(a.z), bf16_lo(b.z), s);
  s = fmaf(bf16_hi(a.z), bf16_hi(b.z), s);
  s = fmaf(bf16_lo(a.w), bf16_lo(b.w), s);
  s = fmaf(bf16_hi(a.w), bf16_hi(b.w), s);
  return s;
}

// T = t + 1 positions, NP = pieces per lane, DH = head size.
template <int T, int NP, int DH>
__global__ void __launch_bounds__(128)
self_attn_kernel(const SelfAttnParams p) {
  pdl_wait();
  pdl_trigger();
  constexpr int kLanesPerHead = DH / 8;
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= p.R) return;
  constexpr int t = T - 1;
  const int M_t = p.beam[t];
  const int b = r / M_t;
  const int pieces = p.HD >> 3;
  const int seg_base = blockIdx.y * (NP * 32);             // first 16-byte piece of this warp's segment

  // own q, k, v
  const uint4* qrow = reinterpret_cast<const uint4*>(p.qkv + (int64_t)r * p.qkv_row_stride);
  uint4 q[NP], kk[T][NP], vv[T][NP];
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const int pc = seg_base + i * 32 + lane;
    if (pc < pieces) {
      q[i] = __ldg(qrow + pc);
      kk[t][i] = __ldg(qrow + pieces + pc);
      vv[t][i] = __ldg(qrow + 2 * pieces + pc);
    } else {
      q[i] = kk[t][i] = vv[t][i] = make_uint4(0, 0, 0, 0);
    }
  }
  // ancestor chain: rows[j] = global row of the prefix token j
  int64_t rows[T];
  {
    int local = r - b * M_t;
    bool bad = false;
#pragma unroll
    for (int j = t; j >= 1; --j) {
      rows[j] = (int64_t)b * p.beam[j] + local;
      int par = __ldg(p.parents + (int64_t)j * p.R_max + rows[j]);
      if (par < 0 || par >= p.beam[j - 1]) { bad = true; par = 0; }
      local = par;
    }
    rows[0] = (int64_t)b * p.beam[0] + local;
    if (bad && lane == 0 && blockIdx.y == 0) flag_status(p.d_status, GRACE_DEV_BAD_INDEX);
  }
  // all prefix loads in flight together
#pragma unroll
  for (int j = 0; j < t; ++j) {
    const int64_t off = (int64_t)j * p.cache_slab_stride + rows[j] * p.cache_row_stride;
    const uint4* kr = reinterpret_cast<const uint4*>(p.k_cache + off);
    const uint4* vr = reinterpret_cast<const uint4*>(p.v_cache + off);
#pragma unroll
    for (int i = 0; i < NP; ++i) {
      const int pc = seg_base + i * 32 + lane;
      if (pc < pieces) { kk[j][i] = __ldg(kr + pc); vv[j][i] = __ldg(vr + pc); }
      else { kk[j][i] = vv[j][i] = make_uint4(0, 0, 0, 0); }
    }
  }
  // cache write of the current token (slab t, this row)
  if (p.write_cache) {
    const int64_t off = (int64_t)t * p.cache_slab_stride + (int64_t)r * p.cache_row_stride;
    uint4* kw = reinterpret_cast<uint4*>(p.k_cache + off);
    uint4* vw = reinterpret_cast<uint4*>(p.v_cache + off);
#pragma unroll
    for (int i = 0; i < NP; ++i) {
      const int pc = seg_base + i * 32 + lane;
      if (pc < pieces) { kw[pc] = kk[t][i]; vw[pc] = vv[t][i]; }
    }
  }
  uint4* orow = reinterpret_cast<uint4*>(p.out + (int64_t)r * p.out_row_stride);
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    float s[T];
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < T; ++j) {
      float d = dot8(q[i], kk[j][i]);
#pragma unroll
      for (int o = 1; o < kLanesPerHead; o <<= 1) d += __shfl_xor_sync(kFullMask, d, o);
      s[j] = d * p.scale;
      mx = fmaxf(mx, s[j]);
    }
    float den = 0.f;
#pragma unroll
    for (int j = 0; j < T; ++j) { s[j] = __expf(s[j] - mx); den += s[j]; }
    const float inv = 1.f / den;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
    for (int j = 0; j < T; ++j) {
      const float w = s[j] * inv;
      const uint4 v = vv[j][i];
      acc[0] = fmaf(w, bf16_lo(v.x), acc[0]); acc[1] = fmaf(w, bf16_hi(v.x), acc[1]);
      acc[2] = fmaf(w, bf16_lo(v.y), acc[2]); acc[3] = fmaf(w, bf16_hi(v.y), acc[3]);
      acc[4] = fmaf(w, bf16_lo(v.z), acc[4]); acc[5] = fmaf(w, bf16_hi(v.z), acc[5]);
      acc[6] = fmaf(w, bf16_lo(v.w), acc[6]); acc[7] = fmaf(w, bf16_hi(v.w), acc[7]);
    }
    const int pc = seg_base + i * 32 + lane;
    if (pc < pieces)
      orow[pc] = make_uint4(pack_bf16x2(acc[0], acc[1]), pack_bf16x2(acc[2], acc[3]),
                            pack_bf16x2(acc[4], acc[5]), pack_bf16x2(acc[6], acc[7]));
  }
}

template <int T, int NP>
static grace_status_t launch_dh(const SelfAttnParams& p, int d_h, cudaStream_t s) {
  const int warps = 4;
  const dim3 blocks((p.R + warps - 1) / warps, (p.HD / 8 + NP * 32 - 1) / (NP * 32));
  switch (d_h) {
    case 32: launch_pdl(self_attn_kernel<T, NP, 32>, blocks, dim3(warps * 32), 0, s, p); break;
    case 64: launch_pdl(self_attn_kernel<T, NP, 64>, blocks, dim3(warps * 32), 0, s, p); break;
    case 128: launch_pdl(self_attn_kernel<T, NP, 128>, blocks, dim3(warps * 32), 0, s, p); break;
    default: return GRACE_UNSUPPORTED_SHAPE;
  }
  GRACE_LAUNCH_CHECK();
  return GRACE_OK;
}

template <int T>
static grace_status_t launch_np(const SelfAttnParams& p, int d_h, cudaStream_t s) {
  const int np = (p.HD / 8 + 31) / 32;
  switch (np) {
    case 1: return launch_dh<T, 1>(p, d_h, s);
    // From four positions on, a row of 64 pieces goes to two warps (32 pieces each): the K / V registers of a
    // thread halve and more warps fit (65536 rows x 512, T_self = 4: 103.7 -> 99.6 us, in place 89.4 -> 85.3;
    // T_self = 5: 124 -> 118); with fewer positions one warp per row is as fast or faster.
    case 2: return (T >= 4) ? launch_dh<T, 1>(p, d_h, s) : launch_dh<T, 2>(p, d_h, s);
    // wider rows: segments of 4 x 32 pieces, one warp each; from three positions on segments of 32 pieces
    // (16384 rows x 2048, in place: T_self = 3: 84.0 -> 80.4 us, T_self = 4: 107.7 -> 93.9 us)
    default: return (T >= 3) ? launch_dh<T, 1>(p, d_h, s) : launch_dh<T, 4>(p, d_h, s);
  }
}

}  // namespace grace

static grace_status_t self_attn_impl(const uint16_t* qkv, int64_t qkv_row_stride, uint16_t* k_cache, uint16_t* v_cache,
                                     int64_t cache_row_stride, int64_t cache_slab_stride, int write_cache,
                                     const int32_t* parents, const int32_t* beam_sizes, uint16_t* out,
                                     int64_t out_row_stride, int B, int t, int H, int d_h, int64_t R_max, float scale,
                                     int32_t* d_status, void* stream) {
  using namespace grace;
  if (!qkv || !k_cache || !v_cache || !beam_sizes || !out || (t > 0 && !parents)) return GRACE_INVALID_ARG;
  if (B <= 0 || H <= 0 || t < 0) return GRACE_INVALID_ARG;
  if (t >= kMaxSelfSteps || (d_h != 32 && d_h != 64 && d_h != 128)) return GRACE_UNSUPPORTED_SHAPE;
  const int HD = H * d_h;
  if (HD > 8192) return GRACE_UNSUPPORTED_SHAPE;
  if (!grace_aligned16(qkv) || !grace_aligned16(k_cache) || !grace_aligned16(v_cache) || !grace_aligned16(out) ||
      (qkv_row_stride & 7) || (out_row_stride & 7) || qkv_row_stride < 3 * HD || out_row_stride < HD ||
      (cache_row_stride & 7) || (cache_slab_stride & 7) || cache_row_stride < HD)
    return GRACE_INVALID_ARG;
  SelfAttnParams p;
  for (int j = 0; j <= t; ++j) {
    if (beam_sizes[j] <= 0 || (int64_t)B * beam_sizes[j] > R_max) return GRACE_INVALID_ARG;
    p.beam[j] = beam_sizes[j];
  }
  p.qkv = qkv; p.k_cache = k_cache; p.v_cache = v_cache; p.parents = parents; p.out = out;
  p.d_status = d_status; p.qkv_row_stride = qkv_row_stride; p.out_row_stride = out_row_stride;
  p.cache_row_stride = cache_row_stride; p.cache_slab_stride = cache_slab_stride; p.write_cache = write_cache;
  p.R_max = R_max; p.R = B * beam_sizes[t]; p.t = t; p.HD = HD; p.scale = scale;
  cudaStream_t s = (cudaStream_t)stream;
  switch (t) {
    case 0: return launch_np<1>(p, d_h, s);
    case 1: return launch_np<2>(p, d_h, s);
    case 2: return launch_np<3>(p, d_h, s);
    case 3: return launch_np<4>(p, d_h, s);
    case 4: return launch_np<5>(p, d_h, s);
    case 5: return launch_np<6>(p, d_h, s);
    case 6: return launch_np<7>(p, d_h, s);
    case 7: return launch_np<8>(p, d_h, s);
  }
  return GRACE_UNSUPPORTED_SHAPE;
}

extern "C" grace_status_t grace_self_attn(const uint16_t* qkv, int64_t qkv_row_stride,
                                          uint16_t* k_cache, uint16_t* v_cache,
                                          const int32_t* parents, const int32_t* beam_sizes,
                                          uint16_t* out, int64_t out_row_stride,
                                          int B, int t, int H, int d_h, int64_t R_max, float scale,
                                          int32_t* d_status, void* stream) {
  const int64_t HD = (int64_t)H * d_h;
  return self_attn_impl(qkv, qkv_row_stride, k_cache, v_cache, HD, R_max * HD, 1, parents, beam_sizes, out,
                        out_row_stride, B, t, H, d_h, R_max, scale, d_status, stream);
}

extern "C" grace_status_t grace_self_attn_inplace(uint16_t* qkv_slabs, int64_t row_stride, int64_t slab_stride,
                                                  const int32_t* parents, const int32_t* beam_sizes,
                                                  uint16_t* out, int64_t out_row_stride,
                                                  int B, int t, int H, int d_h, int64_t R_max, float scale,
                                                  int32_t* d_status, void* stream) {
  if (!qkv_slabs || H <= 0 || t < 0 || slab_stride < R_max * row_stride) return GRACE_INVALID_ARG;
  const int64_t HD = (int64_t)H * d_h;
  return self_attn_impl(qkv_slabs + (int64_t)t * slab_stride, row_stride, qkv_slabs + HD, qkv_slabs + 2 * HD,
                        row_stride, slab_stride, 0, parents, beam_sizes, out, out_row_stride, B, t, H, d_h, R_max,
                        scale, d_status, stream);
}
