// Cross-attention on tcgen05 tensor cores (Section 5.1: beams of a request are the M dimension of
// a dense contraction against that request's shared K/V), head size 64.
//
// One CTA owns 128 query rows of one (request, head) and streams the encoder positions in blocks
// of 128:
//   S   = Q K_blk^T        tcgen05.mma, A = Q (shared, K-major), B = K_blk (shared, K-major),
//                          fp32 S[128 x 128] in TMEM
//   P   = exp2(S*c - max)  128 softmax threads, one query row each (TMEM lane = row); P is
//                          written back over S as packed bf16
//   O_b = P V_blk          tcgen05.mma, A = P (TMEM), B = V_blk (shared, read MN-major, so V is
//                          used as stored: no transpose anywhere)
//   O  += O_b              in registers, with the usual running-max rescale
// K/V blocks arrive by TMA through a two-stage ring; Q, K and V are addressed with 4-D tensor
// maps over the caller's strides, so the beam-major Q / O layout is never permuted (the view /
// permute / reshape chain of Section 5.1 costs nothing).  Ragged M and T are zero-filled by TMA
// and masked in the softmax.  Warp roles: 0-3 softmax + epilogue, 4 TMA producer, 5 MMA issuer.
// Two CTAs share an SM, so one CTA's MMAs run under the other's exponentials.
#pragma once
#include "common.cuh"
#include "tc.cuh"

namespace grace {

constexpr int kCaBM = 128;        // query rows per CTA
constexpr int kCaBN = 128;        // encoder positions per block
constexpr int kCaDH = 64;
constexpr int kCaStages = 2;
constexpr int kCaTileBytes = 128 * 64 * 2;                       // 16 KB: Q, K_blk or V_blk
constexpr int kCaSmemBytes = kCaTileBytes * (1 + 2 * kCaStages) + 1024 + 256;
constexpr uint32_t kCaTmemCols = 256;                            // S/P: 0..127, O_blk: 128..191

struct CrossTcParams {
  uint16_t* out;
  float* lse;
  int64_t out_row_stride;
  int M, H, T;
  float scale_log2;             // scale * log2(e)
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(192)
cross_attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                     const __grid_constant__ CUtensorMap map_v, const CrossTcParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* q_tile = tiles;
  uint8_t* kv_tiles = tiles + kCaTileBytes;                      // stage s: K at 2s, V at 2s+1
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + kCaTileBytes * (1 + 2 * kCaStages));
  uint64_t* q_full = bars;
  uint64_t* kv_full = bars + 1;
  uint64_t* kv_empty = kv_full + kCaStages;
  uint64_t* s_full = kv_empty + kCaStages;
  uint64_t* p_full = s_full + 1;
  uint64_t* o_last = p_full + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_last + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * kCaBM, h = blockIdx.y, b = blockIdx.z;
  const int NB = (p.T + kCaBN - 1) / kCaBN;

  if (threadIdx.x == 0) {
    tc::mbar_init(q_full, 1);
    for (int s = 0; s < kCaStages; ++s) { tc::mbar_init(kv_full + s, 1); tc::mbar_init(kv_empty + s, 1); }
    tc::mbar_init(s_full, 1);
    tc::mbar_init(p_full, 4);                  // one arrival per softmax warp
    tc::mbar_init(o_last, 1);
    *abort_flag = 0;
    tc::fence_mbar_init();
  }
  if (warp == 4) tc::tmem_alloc(tmem_slot, kCaTmemCols);
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_s = tmem_base;           // S fp32 cols 0..127; P bf16x2 cols 0..63
  const uint32_t tmem_o = tmem_base + 128;     // O_blk fp32 cols 128..191

  if (warp == 4) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      tc::tma_prefetch_desc(&map_q); tc::tma_prefetch_desc(&map_k); tc::tma_prefetch_desc(&map_v);
      tc::mbar_expect_tx(q_full, kCaTileBytes);
      tc::tma_load_4d(q_tile, &map_q, q_full, 0, h, m0, b);
      for (int j = 0; j < NB; ++j) {
        const int s = j % kCaStages;
        if (!tc::mbar_wait(kv_empty + s, ((j / kCaStages) & 1) ^ 1, abort_flag)) break;
        tc::mbar_expect_tx(kv_full + s, 2 * kCaTileBytes);
        tc::tma_load_4d(kv_tiles + (2 * s) * kCaTileBytes, &map_k, kv_full + s, 0, j * kCaBN, h, b);
        tc::tma_load_4d(kv_tiles + (2 * s + 1) * kCaTileBytes, &map_v, kv_full + s, 0, j * kCaBN, h, b);
      }
    }
  } else if (warp == 5) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc_s = tc::idesc_bf16(kCaBM, kCaBN, 0);     // Q K^T : B K-major
      constexpr uint32_t idesc_o = tc::idesc_bf16(kCaBM, kCaDH, 1);     // P V   : B MN-major
      const uint32_t q_addr = tc::smem_addr(q_tile);
      bool ok = tc::mbar_wait(q_full, 0, abort_flag) && tc::mbar_wait(kv_full + 0, 0, abort_flag);
      if (ok) {
        tc::tc_fence_after();
        const uint32_t k_addr = tc::smem_addr(kv_tiles);
#pragma unroll
        for (int k = 0; k < kCaDH / 16; ++k)
          tc::mma_ss(tmem_s, tc::smem_desc_sw128(q_addr + 32 * k, 16, 1024),
                     tc::smem_desc_sw128(k_addr + 32 * k, 16, 1024), idesc_s, k ? 1u : 0u);
        tc::mma_commit(s_full);
      }
      for (int j = 0; ok && j < NB; ++j) {
        const int s = j % kCaStages;
        if (!tc::mbar_wait(p_full, j & 1, abort_flag)) break;
        tc::tc_fence_after();
        const uint32_t v_addr = tc::smem_addr(kv_tiles + (2 * s + 1) * kCaTileBytes);
#pragma unroll
        for (int k = 0; k < kCaBN / 16; ++k)
          tc::mma_ts(tmem_o, tmem_s + 8 * k, tc::smem_desc_sw128(v_addr + 2048 * k, 1024, 1024), idesc_o,
                     k ? 1u : 0u);
        tc::mma_commit(kv_empty + s);                       // K_blk, V_blk of block j are consumed
        if (j + 1 < NB) {
          const int s1 = (j + 1) % kCaStages;
          if (!tc::mbar_wait(kv_full + s1, ((j + 1) / kCaStages) & 1, abort_flag)) break;
          tc::tc_fence_after();
          const uint32_t k_addr = tc::smem_addr(kv_tiles + (2 * s1) * kCaTileBytes);
#pragma unroll
          for (int k = 0; k < kCaDH / 16; ++k)
            tc::mma_ss(tmem_s, tc::smem_desc_sw128(q_addr + 32 * k, 16, 1024),
                       tc::smem_desc_sw128(k_addr + 32 * k, 16, 1024), idesc_s, k ? 1u : 0u);
          tc::mma_commit(s_full);                           // also: O_blk of block j is complete
        } else {
          tc::mma_commit(o_last);
        }
      }
    }
  } else {
    // ---------------- softmax + epilogue: thread = query row ----------------
    const int row = warp * 32 + lane;                       // TMEM lane
    const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
    float m_run = -INFINITY, l_run = 0.f;
    float o_acc[kCaDH];
#pragma unroll
    for (int i = 0; i < kCaDH; ++i) o_acc[i] = 0.f;
    bool ok = true;
    for (int j = 0; j < NB; ++j) {
      ok = ok && tc::mbar_wait(s_full, j & 1, abort_flag);
      ok = __all_sync(kFullMask, ok);
      if (!ok) break;
      tc::tc_fence_after();
      if (j > 0) {                                          // O_blk of block j-1 is complete too
#pragma unroll
        for (int c = 0; c < kCaDH / 32; ++c) {
          uint32_t r[32];
          tc::tmem_ld32(tmem_o + lane_addr + 32 * c, r);
          tc::tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) o_acc[32 * c + i] += __uint_as_float(r[i]);
        }
      }
      const int valid = min(kCaBN, p.T - j * kCaBN);        // columns of this block that exist
      // pass 1: row maximum
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < kCaBN / 32; ++c) {
        uint32_t r[32];
        tc::tmem_ld32(tmem_s + lane_addr + 32 * c, r);
        tc::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (32 * c + i < valid) mx = fmaxf(mx, __uint_as_float(r[i]));
      }
      const float m_new = fmaxf(m_run, mx * p.scale_log2);
      const float alpha = ex2(m_run - m_new);               // 0 on the first block
      if (alpha != 1.f) {
        l_run *= alpha;
#pragma unroll
        for (int i = 0; i < kCaDH; ++i) o_acc[i] *= alpha;
      }
      m_run = m_new;
      // pass 2: probabilities, written over S as packed bf16
      float sum = 0.f;
#pragma unroll
      for (int c = 0; c < kCaBN / 32; ++c) {
        uint32_t r[32];
        tc::tmem_ld32(tmem_s + lane_addr + 32 * c, r);
        tc::tmem_ld_wait();
        uint32_t packed[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          float e0 = ex2(fmaf(__uint_as_float(r[2 * i]), p.scale_log2, -m_new));
          float e1 = ex2(fmaf(__uint_as_float(r[2 * i + 1]), p.scale_log2, -m_new));
          if (32 * c + 2 * i >= valid) e0 = 0.f;
          if (32 * c + 2 * i + 1 >= valid) e1 = 0.f;
          sum += e0 + e1;
          packed[i] = pack_bf16x2(e0, e1);
        }
        tc::tmem_st16(tmem_s + lane_addr + 16 * c, packed);
      }
      l_run += sum;
      tc::tmem_st_wait();
      tc::tc_fence_before();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(p_full);
    }
    if (ok) ok = tc::mbar_wait(o_last, 0, abort_flag);
    ok = __all_sync(kFullMask, ok);
    if (ok) {
      tc::tc_fence_after();
#pragma unroll
      for (int c = 0; c < kCaDH / 32; ++c) {
        uint32_t r[32];
        tc::tmem_ld32(tmem_o + lane_addr + 32 * c, r);
        tc::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) o_acc[32 * c + i] += __uint_as_float(r[i]);
      }
      const int m = m0 + row;
      if (m < p.M) {
        const float inv = 1.f / l_run;
        const int64_t r_out = (int64_t)b * p.M + m;
        uint4* dst = reinterpret_cast<uint4*>(p.out + r_out * p.out_row_stride + h * kCaDH);
#pragma unroll
        for (int i = 0; i < kCaDH / 8; ++i)
          dst[i] = make_uint4(pack_bf16x2(o_acc[8 * i] * inv, o_acc[8 * i + 1] * inv),
                              pack_bf16x2(o_acc[8 * i + 2] * inv, o_acc[8 * i + 3] * inv),
                              pack_bf16x2(o_acc[8 * i + 4] * inv, o_acc[8 * i + 5] * inv),
                              pack_bf16x2(o_acc[8 * i + 6] * inv, o_acc[8 * i + 7] * inv));
        if (p.lse != nullptr) p.lse[r_out * p.H + h] = (m_run + log2f(l_run)) * 0.6931471805599453f;
      }
    }
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == 4) tc::tmem_dealloc(tmem_base, kCaTmemCols);
}

inline bool cross_attn_tc_supported(int B, int M, int H, int d_h, int T_ctx) {
  return d_h == kCaDH && H <= 65535 && B <= 65535 && T_ctx >= 1 && M >= 1;
}

inline grace_status_t launch_cross_attn_tc(const uint16_t* q, int64_t q_row_stride, const uint16_t* k,
                                           const uint16_t* v, int64_t kv_stride_b, int64_t kv_stride_h,
                                           int64_t kv_stride_t, uint16_t* out, int64_t out_row_stride, float* lse,
                                           int B, int M, int H, int d_h, int T_ctx, float scale, cudaStream_t s) {
  (void)d_h;
  CUtensorMap mq, mk, mv;
  {
    const uint64_t dims[4] = {(uint64_t)kCaDH, (uint64_t)H, (uint64_t)M, (uint64_t)B};
    const uint64_t str[3] = {(uint64_t)kCaDH, (uint64_t)q_row_stride, (uint64_t)M * (uint64_t)q_row_stride};
    const uint32_t box[4] = {(uint32_t)kCaDH, 1u, (uint32_t)kCaBM, 1u};
    if (!tc::make_tmap_bf16(&mq, q, 4, dims, str, box)) return GRACE_CUDA_ERROR;
  }
  {
    const uint64_t dims[4] = {(uint64_t)kCaDH, (uint64_t)T_ctx, (uint64_t)H, (uint64_t)B};
    const uint64_t str[3] = {(uint64_t)kv_stride_t, (uint64_t)kv_stride_h, (uint64_t)kv_stride_b};
    const uint32_t box[4] = {(uint32_t)kCaDH, (uint32_t)kCaBN, 1u, 1u};
    if (!tc::make_tmap_bf16(&mk, k, 4, dims, str, box)) return GRACE_CUDA_ERROR;
    if (!tc::make_tmap_bf16(&mv, v, 4, dims, str, box)) return GRACE_CUDA_ERROR;
  }
  static bool attr_set = false;
  if (!attr_set) {
    GRACE_CUDA_TRY(cudaFuncSetAttribute(cross_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kCaSmemBytes));
    attr_set = true;
  }
  CrossTcParams p;
  p.out = out; p.lse = lse; p.out_row_stride = out_row_stride; p.M = M; p.H = H; p.T = T_ctx;
  p.scale_log2 = scale * 1.4426950408889634f;
  dim3 grid((unsigned)((M + kCaBM - 1) / kCaBM), (unsigned)H, (unsigned)B);
  cross_attn_tc_kernel<<<grid, 192, kCaSmemBytes, s>>>(mq, mk, mv, p);
  GRACE_LAUNCH_CHECK();
  return GRACE_OK;
}

}  // namespace grace
