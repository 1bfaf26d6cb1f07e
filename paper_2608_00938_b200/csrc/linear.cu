// y = act(x @ w^T) (+ residual): the projection / feed-forward / logits GEMMs of the decoder
// layer (Section 3.2), on tcgen05 tensor cores.
//
// One CTA computes a 128 x BN output tile.  A producer thread streams 128 x 64 bf16 tiles of x
// and BN x 64 tiles of w through a ring of shared-memory stages with TMA (128-byte swizzle,
// out-of-range rows read as zero, so ragged M and N need no special path).  One thread issues
// tcgen05.mma (M = 128, N = BN, K = 16 per instruction) with the fp32 accumulator in TMEM;
// tcgen05.commit frees each stage as soon as the tensor core has consumed it.  All four warps then
// read the accumulator back (each warp its own 32 TMEM lanes = 32 output rows), apply ReLU /
// residual, and store bf16 or fp32.  Two CTAs fit on an SM, so one CTA's epilogue overlaps the
// other's main loop.
#include "common.cuh"
#include "tc.cuh"

namespace grace {
__device__ __forceinline__ float fast_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}


constexpr int kGemmBM = 128;
constexpr int kGemmBK = 64;

// STAGES = 3: throughput form (several CTAs per SM).  STAGES = 8 with BN = 32: latency form for launches whose grid
// does not fill the GPU (step 0 of a decode: 32 rows): the whole K = 512 of a tile is in flight at once, and the
// narrow tile spreads the weight stream over twice as many SMs as BN = 64 did (step 0: 382 -> 352 us; BN = 16: same).
template <int BN, int STAGES>
struct GemmSmem {
  static constexpr int kABytes = kGemmBM * kGemmBK * 2;
  static constexpr int kBBytes = BN * kGemmBK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kTotal = STAGES * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

struct GemmParams {
  uint16_t* y_bf16;
  float* y_f32;
  const float* residual;
  const uint16_t* residual_bf16;   // bf16 residual stream (added in fp32, result rounded to bf16)
  // LayerNorm folded into the GEMM (x is the raw stream, w carries the gain): y = row.x * acc + row.y * col_sum + col_bias
  const float2* aff_row;           // [M]: (rstd, -rstd * mean) of the row; nullptr = plain GEMM
  const float* aff_cs;             // [N]: sum over k of w[n][k]
  const float* aff_cb;             // [N]: sum over k of beta[k] * w0[n][k]
  int64_t ldy;
  int M, N, K, relu;
};

template <int BN, int STAGES>
__global__ void __launch_bounds__(128)
linear_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
              const GemmParams p) {
  // The weights do not depend on the kernel before this one: their first tiles are requested before the wait
  // on that kernel, so their trip from HBM overlaps its tail; every thread waits before its first access to
  // anything an earlier kernel wrote (activations, row statistics, the residual).
  pdl_trigger();
  constexpr int kGemmStages = STAGES;
  using S = GemmSmem<BN, STAGES>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* full = reinterpret_cast<uint64_t*>(tiles + kGemmStages * S::kStageBytes);
  uint64_t* empty = full + kGemmStages;
  uint64_t* accum_bar = empty + kGemmStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum_bar + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.y * kGemmBM, n0 = blockIdx.x * BN;
  const int KB = p.K / kGemmBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kGemmStages; ++s) { tc::mbar_init(full + s, 1); tc::mbar_init(empty + s, 1); }
    tc::mbar_init(accum_bar, 1);
    *abort_flag = 0;
    tc::fence_mbar_init();
    tc::tma_prefetch_desc(&map_x);
    tc::tma_prefetch_desc(&map_w);
  }
  if (warp == 0) tc::tmem_alloc(tmem_slot, BN < 32 ? 32 : BN);
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0 && lane == 0) {
    // ---- TMA producer ----
    const int first = KB < kGemmStages ? KB : kGemmStages;  // the ring's first pass needs no empty-slot wait
    for (int kb = 0; kb < first; ++kb) {
      tc::mbar_expect_tx(full + kb, S::kStageBytes);
      tc::tma_load_2d(tiles + kb * S::kStageBytes + S::kABytes, &map_w, full + kb, kb * kGemmBK, n0);
    }
    pdl_wait();
    for (int kb = 0; kb < first; ++kb)
      tc::tma_load_2d(tiles + kb * S::kStageBytes, &map_x, full + kb, kb * kGemmBK, m0);
    for (int kb = first; kb < KB; ++kb) {
      const int s = kb % kGemmStages;
      if (!tc::mbar_wait(empty + s, ((kb / kGemmStages) & 1) ^ 1, abort_flag)) break;
      tc::mbar_expect_tx(full + s, S::kStageBytes);
      uint8_t* a = tiles + s * S::kStageBytes;
      tc::tma_load_2d(a, &map_x, full + s, kb * kGemmBK, m0);
      tc::tma_load_2d(a + S::kABytes, &map_w, full + s, kb * kGemmBK, n0);
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer ----
    constexpr uint32_t idesc = tc::idesc_bf16(kGemmBM, BN, 0);
    for (int kb = 0; kb < KB; ++kb) {
      const int s = kb % kGemmStages;
      if (!tc::mbar_wait(full + s, (kb / kGemmStages) & 1, abort_flag)) break;
      tc::tc_fence_after();
      const uint32_t a_addr = tc::smem_addr(tiles + s * S::kStageBytes);
      const uint64_t a_desc = tc::smem_desc_sw128(a_addr, 16, 1024);
      const uint64_t b_desc = tc::smem_desc_sw128(a_addr + S::kABytes, 16, 1024);
#pragma unroll
      for (int k = 0; k < kGemmBK / 16; ++k)
        tc::mma_ss(tmem_base, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc, (kb | k) ? 1u : 0u);
      tc::mma_commit(empty + s);
    }
    tc::mma_commit(accum_bar);
  }
  __syncwarp();
  pdl_wait();

  // ---- epilogue: warp w owns TMEM lanes 32w .. 32w+31 = rows m0 + 32w + lane ----
  // Folded LayerNorm: the row's pair and the column vectors of a chunk are fetched (from clamped addresses,
  // unconditionally) one chunk ahead of their use, the first while the accumulator is still filling.
  const bool folded = p.aff_row != nullptr;
  const float* cs_or_cb = p.aff_cs != nullptr ? p.aff_cs : p.aff_cb;
  float2 ar = make_float2(1.f, 0.f);
  float4 cs_next[4], cb_next[4];
  auto fetch_cols = [&](int c) {
    if (!folded) return;
    const int n = min(n0 + c, p.N - 16);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      cb_next[j] = __ldg(reinterpret_cast<const float4*>(p.aff_cb + n) + j);
      cs_next[j] = __ldg(reinterpret_cast<const float4*>(cs_or_cb + n) + j);
    }
  };
  if (folded) ar = __ldg(p.aff_row + min(m0 + warp * 32 + lane, p.M - 1));
  fetch_cols(0);
  const bool ok = tc::mbar_wait(accum_bar, 0, abort_flag);
  tc::tc_fence_after();
  __syncwarp();
  if (ok) {
    const int m = m0 + warp * 32 + lane;
#pragma unroll 1
    for (int c = 0; c < BN; c += 16) {
      uint32_t acc[16];
      tc::tmem_ld16(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c, acc);
      float cs[16], cb[16];
      if (folded) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          cs[4 * j] = cs_next[j].x; cs[4 * j + 1] = cs_next[j].y; cs[4 * j + 2] = cs_next[j].z; cs[4 * j + 3] = cs_next[j].w;
          cb[4 * j] = cb_next[j].x; cb[4 * j + 1] = cb_next[j].y; cb[4 * j + 2] = cb_next[j].z; cb[4 * j + 3] = cb_next[j].w;
        }
        if (c + 16 < BN) fetch_cols(c + 16);
      }
      tc::tmem_ld_wait();
      const int n = n0 + c;
      if (m < p.M && n < p.N) {           // N % 16 == 0: the 16 columns are all in or all out
        float v[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          v[j] = __uint_as_float(acc[j]);
          if (folded) v[j] = fmaf(ar.x, v[j], p.aff_cs != nullptr ? fmaf(ar.y, cs[j], cb[j]) : cb[j]);
          if (p.relu) v[j] = fmaxf(v[j], 0.f);
        }
        if (p.residual != nullptr) {
          const float4* res = reinterpret_cast<const float4*>(p.residual + (int64_t)m * p.ldy + n);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float4 r4 = res[j];
            v[4 * j] += r4.x; v[4 * j + 1] += r4.y; v[4 * j + 2] += r4.z; v[4 * j + 3] += r4.w;
          }
        }
        if (p.residual_bf16 != nullptr) {
          const uint4* res = reinterpret_cast<const uint4*>(p.residual_bf16 + (int64_t)m * p.ldy + n);
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const uint4 r4 = res[j];
            v[8 * j] += bf16_lo(r4.x); v[8 * j + 1] += bf16_hi(r4.x); v[8 * j + 2] += bf16_lo(r4.y); v[8 * j + 3] += bf16_hi(r4.y);
            v[8 * j + 4] += bf16_lo(r4.z); v[8 * j + 5] += bf16_hi(r4.z); v[8 * j + 6] += bf16_lo(r4.w); v[8 * j + 7] += bf16_hi(r4.w);
          }
        }
        if (p.y_f32 != nullptr) {
          float4* dst = reinterpret_cast<float4*>(p.y_f32 + (int64_t)m * p.ldy + n);
#pragma unroll
          for (int j = 0; j < 4; ++j) dst[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
        } else {
          uint4* dst = reinterpret_cast<uint4*>(p.y_bf16 + (int64_t)m * p.ldy + n);
          dst[0] = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
          dst[1] = make_uint4(pack_bf16x2(v[8], v[9]), pack_bf16x2(v[10], v[11]), pack_bf16x2(v[12], v[13]), pack_bf16x2(v[14], v[15]));
        }
      }
    }
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tmem_base, BN < 32 ? 32 : BN);
}

// ---------------------------------------------------------------------------------------------
// Persistent CTA-pair kernel for the large GEMMs of the decoder (M in the tens of thousands).
//
// A cluster of two CTAs (two SMs) walks over 256 x 256 output tiles (n fastest, so the pairs running
// at the same time share an A row panel in L2) with one tcgen05.mma.cta_group::2 stream.  Each CTA
// stages its own 128 rows of A and its own 128 rows of W (half of the tile's N) through a 6-stage
// ring, so an SM pulls 32 KB per 64-wide k-block through its port to the L2 where a lone 128 x 256 tile
// needs 48 KB: that port (about 64 bytes per clock for loads and stores together), not the tensor pipe, is
// what limits these GEMMs at K = 512 (256 KB of operands in, 64 KB of bf16 results out per tile and CTA
// against 4096 clocks of MMAs).  The even
// CTA issues every MMA into one of TWO TMEM accumulators (2 x 256 columns = all of TMEM), so the
// four epilogue warps of each CTA drain tile i while the tensor cores already work on tile i+1.
// tcgen05.commit arrives on the barriers of both CTAs, and both CTAs' TMA loads count their bytes on
// the even CTA's "stage full" barrier (plain loads, each with one destination).
// The epilogue reads 64 (bf16) or 32 (fp32) columns at a time from TMEM, writes them to a
// 128-byte-swizzled staging tile in shared memory and hands it to TMA: a plain tile store, or an
// add-reduction straight into the residual stream (x += y), so the residual is never read into the SM.
// ---------------------------------------------------------------------------------------------
constexpr int kPBK = 64;
constexpr int kPStagingBytes = 128 * 128;                 // 128 rows x 128 bytes

enum { kOutBf16 = 0, kOutF32 = 1, kOutF32Add = 2, kOutBf16Add = 3, kOutF32Lse = 4, kOutF32LseAllowed = 5 };

constexpr int kQStages = 6;
constexpr int kQABytes = 128 * kPBK * 2;                  // 16 KB: 128 rows of A
constexpr int kQBBytes = 128 * kPBK * 2;                  // 16 KB: 128 of the tile's 256 rows of W
constexpr int kQStageBytes = kQABytes + kQBBytes;
constexpr int kQAffBytes = 256 * 2 * 4;                   // the tile's 256 (col_sum, col_bias) pairs
// no slack for rounding the base up: the dynamic shared memory is declared 1024-byte aligned and the kernel
// checks it (six stages, the staging buffers and the column vectors leave less than 1 KB of the 227 KB)
constexpr int kQSmem = kQStages * kQStageBytes + 2 * kPStagingBytes + 256 + kQAffBytes;

// STATS: the rows' LayerNorm statistics are not read from memory (aff_row is only a non-null marker then) but
// formed inside the kernel: four more warps per CTA read every A tile out of the ring while the tensor cores
// work on it (a row per thread, its sum and sum of squares over the whole K = the LayerNorm width), and hand
// (rstd, -rstd * mean) of the CTA's 128 rows to the epilogue through 1 KB of shared memory.  A stage is
// released by the MMAs' commit AND by these warps; the odd CTA, whose tiles are counted on the even CTA's
// barrier, learns that a stage has landed from an arrive the even CTA forwards.  Centred rows only (aff_cs ==
// nullptr): the second half of the column-vector buffer is what holds the statistics.
// Log-sum-exp partial of a row over a 256-column tile, 32 columns at a time: running maximum and sum of
// 2^((v - maximum) log2 e).  The tile is summed as TWO halves of 128 columns that are merged at the end: in the
// allowed-only epilogue two threads (of two warp groups) take a half each, elsewhere one thread takes both, and
// both forms give the same bits.
__device__ __forceinline__ void lse_add_chunk(const uint32_t (&r)[32], float& lse_m, float& lse_s) {
  float m0c = fmaxf(__uint_as_float(r[0]), __uint_as_float(r[1])), m1c = fmaxf(__uint_as_float(r[2]), __uint_as_float(r[3]));
#pragma unroll
  for (int i = 4; i < 32; i += 4) {
    m0c = fmaxf(m0c, fmaxf(__uint_as_float(r[i]), __uint_as_float(r[i + 1])));
    m1c = fmaxf(m1c, fmaxf(__uint_as_float(r[i + 2]), __uint_as_float(r[i + 3])));
  }
  const float m_new = fmaxf(lse_m, fmaxf(m0c, m1c));
  const float kLog2e = 1.4426950408889634f;
  const float neg = __fmul_rn(-m_new, kLog2e);
  float s0 = 0.f, s1 = 0.f;
#pragma unroll
  for (int i = 0; i < 32; i += 2) {
    s0 = __fadd_rn(s0, fast_ex2(__fmaf_rn(__uint_as_float(r[i]), kLog2e, neg)));
    s1 = __fadd_rn(s1, fast_ex2(__fmaf_rn(__uint_as_float(r[i + 1]), kLog2e, neg)));
  }
  // first chunk: lse_s = 0 and the factor is 2^-inf = 0
  lse_s = __fmaf_rn(lse_s, fast_ex2(__fmul_rn(__fsub_rn(lse_m, m_new), kLog2e)), __fadd_rn(s0, s1));
  lse_m = m_new;
}
__device__ __forceinline__ float2 lse_merge_halves(float m_a, float s_a, float m_b, float s_b) {
  const float kLog2e = 1.4426950408889634f;
  const float m = fmaxf(m_a, m_b);
  const float ea = fast_ex2(__fmul_rn(__fsub_rn(m_a, m), kLog2e)), eb = fast_ex2(__fmul_rn(__fsub_rn(m_b, m), kLog2e));
  return make_float2(m, __fmaf_rn(s_a, ea, __fmul_rn(s_b, eb)));
}

template <int OUT, bool STATS>
__global__ void __launch_bounds__((STATS || OUT == kOutF32LseAllowed) ? 320 : 192, 1)
linear_pair_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                   const __grid_constant__ CUtensorMap map_y, int M, int N, int K, int relu, float2* lse_part,
                   const float2* __restrict__ aff_row, const float* __restrict__ aff_cs,
                   const float* __restrict__ aff_cb, float ln_eps, const uint64_t* __restrict__ allow_bits,
                   float* __restrict__ y_direct, int64_t ldy) {
  // kOutF32LseAllowed: the log-sum-exp partials of every row and tile as in kOutF32Lse, but of the values
  // themselves only those whose bit is set in allow_bits [M][N / 64] are stored, by the row's own thread at
  // their place in y_direct [M][ldy] (no staging tile, no TMA store): with a constrained decode's allow bits
  // the fp32 logits tensor is never written out.
  extern __shared__ __align__(1024) uint8_t smem_pair[];
  uint8_t* tiles = smem_pair;
  if ((tc::smem_addr(tiles) & 1023u) != 0) {               // the swizzled tiles need it; same answer in every thread
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicAdd(&tc::g_tc_timeouts, 1);
    return;
  }
  uint8_t* staging = tiles + kQStages * kQStageBytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(staging + 2 * kPStagingBytes);   // even CTA only: both CTAs' bytes landed
  uint64_t* empty = full + kQStages;           // the pair's MMAs have read the stage
  uint64_t* acc_full = empty + kQStages;       // [2]
  uint64_t* acc_empty = acc_full + 2;          // [2] even CTA only: 4 local + 4 remote epilogue warps
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  uint64_t* a_ready = acc_empty + 3;           // [kQStages] STATS, odd CTA: the stage has landed (forwarded by the even CTA)
  uint64_t* stats_full = a_ready + kQStages;   // [1] STATS: the tile's row statistics are in shared memory
  uint64_t* stats_empty = stats_full + 1;      // [1] STATS: the epilogue has taken them
  float4* aff_s = reinterpret_cast<float4*>(staging + 2 * kPStagingBytes + 256);   // [128]: (cs, cs, cb, cb) of 2 columns
  float2* stats_s = reinterpret_cast<float2*>(staging + 2 * kPStagingBytes + 256 + kQAffBytes / 2);   // [128] STATS

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = tc::cluster_cta_rank();            // 0: issues the MMAs; 1: peer
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int KB = K / kPBK;
  const int n_tiles = (N + 255) / 256, m_tiles = (M + 255) / 256;
  const int total = n_tiles * m_tiles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kQStages; ++s) { tc::mbar_init(full + s, 1); tc::mbar_init(empty + s, STATS ? 5 : 1); }
    for (int a = 0; a < 2; ++a) { tc::mbar_init(acc_full + a, 1); tc::mbar_init(acc_empty + a, OUT == kOutF32LseAllowed ? 16 : 8); }
    if (STATS) {
      for (int s = 0; s < kQStages; ++s) tc::mbar_init(a_ready + s, 1);
      tc::mbar_init(stats_full, 4);
      tc::mbar_init(stats_empty, 4);
    }
    *abort_flag = 0;
    tc::fence_mbar_init();
    tc::tma_prefetch_desc(&map_x); tc::tma_prefetch_desc(&map_w); tc::tma_prefetch_desc(&map_y);
  }
  if (warp == 0) tc::tmem_alloc_pair(tmem_slot, 512);
  tc::tc_fence_before();
  __syncthreads();
  tc::cluster_sync_all();                                  // both CTAs' barriers exist before any remote arrive
  tc::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();                                              // everything above overlapped the previous kernel's tail
  pdl_trigger();

  if (warp == 0) {
    if (lane == 0) {                                        // ---- TMA producer (both CTAs) ----
      int it = 0;
      for (int tile = pair; tile < total; tile += n_pairs) {
        const int m0 = (tile / n_tiles) * 256 + (int)rank * 128, n0 = (tile % n_tiles) * 256 + (int)rank * 128;
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const int s = it % kQStages;
          if (!tc::mbar_wait_cluster(empty + s, ((it / kQStages) & 1) ^ 1, abort_flag)) { tile = total; break; }
          if (rank == 0) tc::mbar_expect_tx(full + s, 2 * kQStageBytes);     // this CTA's bytes and the peer's
          uint8_t* a = tiles + s * kQStageBytes;
          const uint32_t bar = tc::cluster_addr_of(full + s, 0);
          tc::tma_load_2d_pair(a, &map_x, bar, kb * kPBK, m0);
          tc::tma_load_2d_pair(a + kQABytes, &map_w, bar, kb * kPBK, n0);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {                           // ---- even CTA: MMA issuer for the pair ----
      constexpr uint32_t idesc = tc::idesc_bf16(256, 256, 0);
      int it = 0, local = 0;
      for (int tile = pair; tile < total; tile += n_pairs, ++local) {
        const int ab = local & 1;
        if (!tc::mbar_wait_cluster(acc_empty + ab, ((local >> 1) & 1) ^ 1, abort_flag)) break;
        tc::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(ab * 256);
        bool ok = true;
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const int s = it % kQStages;
          const uint32_t ph = (it / kQStages) & 1;
          if (!tc::mbar_wait_cluster(full + s, ph, abort_flag)) { ok = false; break; }
          tc::tc_fence_after();
          const uint32_t a_addr = tc::smem_addr(tiles + s * kQStageBytes);
          const uint64_t a_desc = tc::smem_desc_sw128(a_addr, 16, 1024);
          const uint64_t b_desc = tc::smem_desc_sw128(a_addr + kQABytes, 16, 1024);
#pragma unroll
          for (int k = 0; k < kPBK / 16; ++k)
            tc::mma_ss_pair(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc, (kb | k) ? 1u : 0u);
          tc::mma_commit_pair(empty + s, 3);
        }
        if (!ok) break;
        tc::mma_commit_pair(acc_full + ab, 3);
      }
    }
  } else if (STATS && warp >= 6) {
    // ---- statistics warps 6..9 of both CTAs: row (warp - 6) * 32 + lane of this CTA's 128 ----
    const int row = (warp - 6) * 32 + lane;
    const float inv_k = 1.f / (float)K;
    int it = 0, local = 0;
    bool ok = true;
    for (int tile = pair; tile < total && ok; tile += n_pairs, ++local) {
      f32x2_t acc = f2_pack(0.f, 0.f), sq = f2_pack(0.f, 0.f);
      for (int kb = 0; kb < KB; ++kb, ++it) {
        const int s = it % kQStages;
        const uint32_t ph = (it / kQStages) & 1;
        if (rank == 0) {
          ok = tc::mbar_wait_cluster(full + s, ph, abort_flag);
          if (ok && warp == 6 && lane == 0) tc::mbar_arrive_remote(a_ready + s, 1);
        } else {
          ok = tc::mbar_wait_cluster(a_ready + s, ph, abort_flag);
        }
        ok = __all_sync(kFullMask, ok);
        if (!ok) break;
        // 128 bytes of the row, in the order that keeps eight neighbouring rows on different banks
        const uint4* a_row = reinterpret_cast<const uint4*>(tiles + s * kQStageBytes + row * 128);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint4 t = a_row[j ^ (row & 7)];
          const f32x2_t a = f2_from_bf16x2(t.x), b = f2_from_bf16x2(t.y), c = f2_from_bf16x2(t.z), d = f2_from_bf16x2(t.w);
          acc = f2_add(acc, f2_add(f2_add(a, b), f2_add(c, d)));
          sq = f2_fma(a, a, sq); sq = f2_fma(b, b, sq); sq = f2_fma(c, c, sq); sq = f2_fma(d, d, sq);
        }
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(empty + s);
      }
      if (!ok) break;
      float lo, hi, qlo, qhi;
      f2_unpack(acc, lo, hi);
      f2_unpack(sq, qlo, qhi);
      const float mean = (lo + hi) * inv_k;
      const float var = fmaxf((qlo + qhi) * inv_k - mean * mean, 0.f);
      const float rstd = rsqrtf(var + ln_eps);
      ok = tc::mbar_wait_cluster(stats_empty, (local & 1) ^ 1, abort_flag);   // the previous tile's were taken
      ok = __all_sync(kFullMask, ok);
      if (!ok) break;
      stats_s[row] = make_float2(rstd, -rstd * mean);
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(stats_full);
    }
  } else {
    // ---- epilogue warps 2..5 of both CTAs: TMEM lane quarter q = rows q*32 + lane of this CTA's 128 ----
    // (kOutF32LseAllowed: warps 6..9 as well; a row's two threads take 128 of the tile's 256 columns each)
    const int q = warp & 3;
    const int half = (warp >= 6) ? 1 : 0;
    const int row = q * 32 + lane;
    const bool issuer = (warp == 2 && lane == 0);
    constexpr bool kBf16Out = (OUT == kOutBf16 || OUT == kOutBf16Add);
    constexpr int kColsPerChunk = kBf16Out ? 64 : 32;
    int local = 0, g = 0;
    // LayerNorm folded into the GEMM: y = ar.x * acc + (ar.y * col_sum + col_bias).  The tile's column vectors go
    // through shared memory (every thread needs all 256 of them); they and the row's pair are fetched one tile
    // ahead, so their latency never sits between two tiles of an epilogue that is the pair's critical path.
    // (The loads are unconditional, from clamped addresses, so that nothing waits for them before their use.)
    float2 ar_next = make_float2(1.f, 0.f), cs_next = make_float2(0.f, 0.f), cb_next = make_float2(0.f, 0.f);
    constexpr bool kAllowed = (OUT == kOutF32LseAllowed);
    ulonglong2 aw_lo_next = make_ulonglong2(0ull, 0ull), aw_hi_next = aw_lo_next;      // the row's 256 allow bits of the tile
    const float* cs_or_cb = aff_cs != nullptr ? aff_cs : aff_cb;
    auto fetch_affine = [&](int tile) {
      if (kAllowed) {
        const int ta = min(tile, total - 1);
        const int ma = (ta / n_tiles) * 256 + (int)rank * 128 + row, na = (ta % n_tiles) * 256;
        const ulonglong2* aw = reinterpret_cast<const ulonglong2*>(allow_bits + (int64_t)min(ma, M - 1) * (N >> 6) + (na >> 6));
        aw_lo_next = __ldg(aw);
        aw_hi_next = __ldg(aw + 1);
        if (ma >= M) aw_lo_next = aw_hi_next = make_ulonglong2(0ull, 0ull);
      }
      if (aff_row == nullptr) return;
      tile = min(tile, total - 1);
      const int m0 = (tile / n_tiles) * 256 + (int)rank * 128, n0 = (tile % n_tiles) * 256;
      const int col = min(n0 + 2 * row, N - 2);
      if (!STATS) ar_next = __ldg(aff_row + min(m0 + row, M - 1));
      cb_next = __ldg(reinterpret_cast<const float2*>(aff_cb + col));
      cs_next = __ldg(reinterpret_cast<const float2*>(cs_or_cb + col));
    };
    fetch_affine(pair);
    for (int tile = pair; tile < total; tile += n_pairs, ++local) {
      const int m0 = (tile / n_tiles) * 256 + (int)rank * 128, n0 = (tile % n_tiles) * 256;
      const int ab = local & 1;
      float2 ar = ar_next;                                 // rows and columns past the edge: values never stored
      const ulonglong2 aw_lo = aw_lo_next, aw_hi = aw_hi_next;
      const float4 cv = aff_cs != nullptr ? make_float4(cs_next.x, cs_next.y, cb_next.x, cb_next.y)
                                          : make_float4(cb_next.x, cb_next.y, 0.f, 0.f);
      bool ok = tc::mbar_wait_cluster(acc_full + ab, (local >> 1) & 1, abort_flag);
      ok = __all_sync(kFullMask, ok);
      if (!ok) break;
      tc::tc_fence_after();
      if (STATS) {
        ok = tc::mbar_wait_cluster(stats_full, local & 1, abort_flag);
        ok = __all_sync(kFullMask, ok);
        if (!ok) break;
        ar = stats_s[row];
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(stats_empty);
      }
      const uint32_t t_acc = tmem_base + (uint32_t)(ab * 256) + ((uint32_t)(q * 32) << 16);
      float lse_m = -INFINITY, lse_s = 0.f;                // kOutF32Lse: running maximum and sum of 2^((v - max) log2 e)
      float lse_m_a = -INFINITY, lse_s_a = 0.f;            //   of the tile's first 128 columns, once the second half has begun
      // read after the first chunk's barrier; the previous tile's readers are past its last barrier.
      // With col_sum: [128] x (cs, cs, cb, cb) of two columns; without: col_bias alone, [256] floats.
      if (aff_row != nullptr && half == 0) {
        if (aff_cs != nullptr) aff_s[row] = cv;
        else reinterpret_cast<float2*>(aff_s)[row] = make_float2(cv.x, cv.y);
      }
      fetch_affine(tile + n_pairs);
      const f32x2_t ar_x = f2_pack(ar.x, ar.x), ar_y = f2_pack(ar.y, ar.y);
      auto fold = [&](uint32_t (&r)[32], int col0) {        // col0: first of the 32 columns, within the tile
        if (aff_row == nullptr) return;
        if (aff_cs == nullptr) {                            // centred rows: y = ar.x * acc + col_bias
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            const float4 c = aff_s[(col0 + i) >> 2];
            float a0, a1, a2, a3;
            f2_unpack(f2_fma(ar_x, f2_pack(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), f2_pack(c.x, c.y)), a0, a1);
            f2_unpack(f2_fma(ar_x, f2_pack(__uint_as_float(r[i + 2]), __uint_as_float(r[i + 3])), f2_pack(c.z, c.w)), a2, a3);
            r[i] = __float_as_uint(a0); r[i + 1] = __float_as_uint(a1);
            r[i + 2] = __float_as_uint(a2); r[i + 3] = __float_as_uint(a3);
          }
          return;
        }
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const float4 c = aff_s[(col0 + i) >> 1];
          const f32x2_t v = f2_fma(ar_x, f2_pack(__uint_as_float(r[i]), __uint_as_float(r[i + 1])),
                                   f2_fma(ar_y, f2_pack(c.x, c.y), f2_pack(c.z, c.w)));
          float lo, hi;
          f2_unpack(v, lo, hi);
          r[i] = __float_as_uint(lo);
          r[i + 1] = __float_as_uint(hi);
        }
      };
      if (kAllowed) {
        // Two threads per row, 128 columns each; no staging tile, no TMA store.  The tile's column vectors in
        // shared memory (written above by the first warp group) are ordered against their readers by the two
        // barriers, which also carry the second half's partial to the thread that merges and stores it.
        tc::named_bar_sync(1, 256);
        const bool sector_aligned = ((reinterpret_cast<uintptr_t>(y_direct) | (uintptr_t)(ldy * 4)) & 31) == 0;
#pragma unroll 1
        for (int cc = 0; cc < 4; ++cc) {
          const int c = half * 4 + cc;
          uint32_t r[32];
          tc::tmem_ld32(t_acc + (uint32_t)(c * 32), r);
          tc::tmem_ld_wait();
          fold(r, c * 32);
          lse_add_chunk(r, lse_m, lse_s);
          const uint64_t aw = half ? ((cc < 2) ? aw_hi.x : aw_hi.y) : ((cc < 2) ? aw_lo.x : aw_lo.y);
          const uint32_t bits = (uint32_t)(aw >> ((c & 1) * 32));
          if (bits != 0u) {
            // whole 32-byte sectors (8 columns) that hold an allowed column: a sector written in full costs the
            // memory system less than a few of its words (no merge with the old contents), and eight predicated
            // stores per chunk instead of thirty-two (measured at 5 % allowed: 173 -> see the notes)
            float* dst = y_direct + (int64_t)(m0 + row) * ldy + n0 + c * 32;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              if ((bits >> (8 * j)) & 0xffu) {
                const uint4 lo = make_uint4(r[8 * j], r[8 * j + 1], r[8 * j + 2], r[8 * j + 3]);
                const uint4 hi = make_uint4(r[8 * j + 4], r[8 * j + 5], r[8 * j + 6], r[8 * j + 7]);
                if (sector_aligned) {
                  st_global_32B(dst + 8 * j, lo, hi);
                } else {
                  *reinterpret_cast<uint4*>(dst + 8 * j) = lo;
                  *reinterpret_cast<uint4*>(dst + 8 * j + 4) = hi;
                }
              }
            }
          }
        }
        float2* part_s = reinterpret_cast<float2*>(staging);       // [128]: the staging tiles are unused here
        if (half == 1) part_s[row] = make_float2(lse_m, lse_s);
        tc::tc_fence_before();
        tc::named_bar_sync(1, 256);
        if (half == 0 && m0 + row < M) {
          const float2 other = part_s[row];
          lse_part[(int64_t)(m0 + row) * n_tiles + (tile % n_tiles)] = lse_merge_halves(lse_m, lse_s, other.x, other.y);
        }
        __syncwarp();
        if (lane == 0) {
          if (rank == 0) tc::mbar_arrive(acc_empty + ab);
          else tc::mbar_arrive_remote(acc_empty + ab, 0);
        }
        continue;
      }
#pragma unroll 1
      for (int c = 0; c < 256 / kColsPerChunk; ++c, ++g) {
        uint8_t* buf = staging + (g & 1) * kPStagingBytes;
        uint32_t rr[kBf16Out ? 2 : 1][32];
        if (kBf16Out) {                                    // the chunk's loads fly while the staging buffer frees up
          tc::tmem_ld32(t_acc + (uint32_t)(c * 64), rr[0]);
          tc::tmem_ld32(t_acc + (uint32_t)(c * 64 + 32), rr[kBf16Out ? 1 : 0]);
        } else {
          tc::tmem_ld32(t_acc + (uint32_t)(c * 32), rr[0]);
        }
        if (issuer) tc::bulk_wait_read<1>();               // the store that last used `buf` has read it
        tc::named_bar_sync(1, 128);
        tc::tmem_ld_wait();
        uint4* my_row = reinterpret_cast<uint4*>(buf + row * 128);
        if (kBf16Out) {
#pragma unroll
          for (int hseg = 0; hseg < 2; ++hseg) {
            uint32_t (&r)[32] = rr[kBf16Out ? hseg : 0];
            fold(r, c * 64 + hseg * 32);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              float v[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                v[e] = __uint_as_float(r[8 * j + e]);
                if (relu) v[e] = fmaxf(v[e], 0.f);
              }
              const int piece = hseg * 4 + j;
              my_row[piece ^ (row & 7)] = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]),
                                                     pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
            }
          }
        } else {
          uint32_t (&r)[32] = rr[0];
          fold(r, c * 32);
          if (OUT == kOutF32Lse) {
            // the row's log-sum-exp over this tile's 256 columns, as two halves of 128 (the tiles of a row are merged later)
            if (c == 4) { lse_m_a = lse_m; lse_s_a = lse_s; lse_m = -INFINITY; lse_s = 0.f; }
            lse_add_chunk(r, lse_m, lse_s);
          }
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            float v[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              v[e] = __uint_as_float(r[4 * j + e]);
              if (relu) v[e] = fmaxf(v[e], 0.f);
            }
            my_row[j ^ (row & 7)] = make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]),
                                               __float_as_uint(v[3]));
          }
        }
        if (c == 256 / kColsPerChunk - 1) {                // accumulator fully read: hand it back to the issuer
          if (OUT == kOutF32Lse && m0 + row < M)
            lse_part[(int64_t)(m0 + row) * n_tiles + (tile % n_tiles)] = lse_merge_halves(lse_m_a, lse_s_a, lse_m, lse_s);
          tc::tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            if (rank == 0) tc::mbar_arrive(acc_empty + ab);
            else tc::mbar_arrive_remote(acc_empty + ab, 0);
          }
        }
        tc::fence_proxy_async_smem();
        tc::named_bar_sync(1, 128);
        if (issuer && m0 < M) {
          if (OUT == kOutF32Add || OUT == kOutBf16Add) tc::tma_reduce_add_2d(&map_y, buf, n0 + c * kColsPerChunk, m0);
          else tc::tma_store_2d(&map_y, buf, n0 + c * kColsPerChunk, m0);
        }
        if (issuer) tc::bulk_commit();
      }
    }
    if (issuer) tc::bulk_wait_all();
  }
  // neither CTA may leave while its peer can still read its shared memory or arrive on its barriers
  tc::tc_fence_before();
  __syncthreads();
  tc::cluster_sync_all();
  if (warp == 0) tc::tmem_dealloc_pair(tmem_base, 512);
}

struct Affine {                                            // LayerNorm folded into the GEMM; row == nullptr: off
  const float2* row;
  const float* cs;
  const float* cb;
  float eps = 0.f;                                         // in_kernel_stats only
  bool in_kernel_stats = false;                            // the pair kernel forms (rstd, -rstd * mean) itself
};
struct AllowedStores {                                     // kOutF32LseAllowed
  const uint64_t* bits = nullptr;
  float* y = nullptr;
  int64_t ldy = 0;
};

template <int OUT, bool STATS = false>
static grace_status_t launch_pair(const CUtensorMap& mx, const CUtensorMap& mw, const CUtensorMap& my, int M, int N,
                                  int K, int relu, cudaStream_t s, float2* lse_part = nullptr,
                                  Affine aff = Affine{nullptr, nullptr, nullptr}, AllowedStores al = AllowedStores{}) {
  static unsigned long long attr_set_devices = 0;
  static int max_clusters_of[kMaxDevices] = {0};
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.blockDim = dim3((STATS || OUT == kOutF32LseAllowed) ? 320 : 192); cfg.dynamicSmemBytes = kQSmem; cfg.stream = s; cfg.attrs = attr; cfg.numAttrs = 2;
  DeviceSetup su(&attr_set_devices);
  if (su) {
    GRACE_CUDA_TRY(cudaFuncSetAttribute(linear_pair_kernel<OUT, STATS>, cudaFuncAttributeMaxDynamicSharedMemorySize, kQSmem));
    int n_sm = 0, clusters = 0;
    GRACE_CUDA_TRY(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, su.dev));
    cfg.gridDim = dim3(n_sm & ~1);
    GRACE_CUDA_TRY(cudaOccupancyMaxActiveClusters(&clusters, linear_pair_kernel<OUT, STATS>, &cfg));
    if (clusters <= 0) return GRACE_CUDA_ERROR;
    if (clusters > n_sm / 2) clusters = n_sm / 2;
    max_clusters_of[su.dev] = clusters;
    su.done();
  }
  const int max_clusters = max_clusters_of[su.dev];
  const int total = ((N + 255) / 256) * ((M + 255) / 256);
  cfg.gridDim = dim3(2 * (total < max_clusters ? total : max_clusters));
  GRACE_CUDA_TRY(cudaLaunchKernelEx(&cfg, linear_pair_kernel<OUT, STATS>, mx, mw, my, M, N, K, relu, lse_part, aff.row, aff.cs, aff.cb, aff.eps,
                                    al.bits, al.y, al.ldy));
  GRACE_LAUNCH_CHECK();
  return GRACE_OK;
}

template <int BN, int STAGES>
static grace_status_t launch_linear(const CUtensorMap& mx, const CUtensorMap& mw, const GemmParams& p, cudaStream_t s) {
  static unsigned long long attr_set_devices = 0;
  DeviceSetup su(&attr_set_devices);
  if (su) {
    GRACE_CUDA_TRY(cudaFuncSetAttribute(linear_kernel<BN, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        GemmSmem<BN, STAGES>::kTotal));
    su.done();
  }
  dim3 grid((p.N + BN - 1) / BN, (p.M + kGemmBM - 1) / kGemmBM);
  launch_pdl(linear_kernel<BN, STAGES>, grid, dim3(128), GemmSmem<BN, STAGES>::kTotal, s, mx, mw, p);
  GRACE_LAUNCH_CHECK();
  return GRACE_OK;
}

}  // namespace grace

static grace_status_t linear_impl(const uint16_t* x, int64_t ldx, const uint16_t* w, int64_t ldw,
                                  uint16_t* y_bf16, float* y_f32, int64_t ldy, const float* residual,
                                  bool add_into_bf16, int M, int N, int K, int relu, void* stream,
                                  float* lse_part = nullptr,
                                  grace::Affine aff = grace::Affine{nullptr, nullptr, nullptr},
                                  const uint64_t* allow_bits = nullptr) {
  using namespace grace;
  if (!x || !w || ((y_bf16 == nullptr) == (y_f32 == nullptr))) return GRACE_INVALID_ARG;
  if (M <= 0 || N <= 0 || K <= 0) return GRACE_INVALID_ARG;
  if ((K % kGemmBK) || (N % 16)) return GRACE_UNSUPPORTED_SHAPE;
  if (!grace_aligned16(x) || !grace_aligned16(w) || !grace_aligned16(y_bf16) || !grace_aligned16(y_f32) ||
      !grace_aligned16(residual) || (ldx & 7) || (ldw & 7) || (ldy & 7) || ldx < K || ldw < K || ldy < N)
    return GRACE_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  const bool aliased = (residual != nullptr) && (residual == y_f32);
  if (lse_part != nullptr && !(M >= 1024 && N >= 256 && (N % 256) == 0 && y_f32 != nullptr && residual == nullptr && !relu))
    return GRACE_UNSUPPORTED_SHAPE;
  if (allow_bits != nullptr && (lse_part == nullptr || (reinterpret_cast<uintptr_t>(allow_bits) & 15)))
    return GRACE_UNSUPPORTED_SHAPE;                          // allowed-only stores exist in the large-problem kernel only
  if (M >= 1024 && N >= 256 && (residual == nullptr || aliased)) {
    // large GEMM: persistent CTA-pair kernel, TMA-store epilogue (add-reduction when y is the residual stream)
    CUtensorMap mx, mw, my;
    const uint64_t dx[2] = {(uint64_t)K, (uint64_t)M}, sx[1] = {(uint64_t)ldx};
    const uint32_t bx[2] = {(uint32_t)kPBK, 128u};
    const uint64_t dw[2] = {(uint64_t)K, (uint64_t)N}, sw[1] = {(uint64_t)ldw};
    const uint32_t bw[2] = {(uint32_t)kPBK, 128u};      // each CTA of a pair stages 128 of the tile's 256 rows of W
    const uint64_t dy[2] = {(uint64_t)N, (uint64_t)M}, sy[1] = {(uint64_t)ldy};
    const bool f32 = (y_f32 != nullptr);
    const uint32_t by[2] = {f32 ? 32u : 64u, 128u};
    if (!tc::make_tmap_bf16(&mx, x, 2, dx, sx, bx) || !tc::make_tmap_bf16(&mw, w, 2, dw, sw, bw) ||
        !tc::make_tmap(&my, f32 ? (const void*)y_f32 : (const void*)y_bf16, 2, dy, sy, by, f32))
      return GRACE_CUDA_ERROR;
    if (aff.row != nullptr && (add_into_bf16 || aliased)) return GRACE_INVALID_ARG;
    if (allow_bits != nullptr)
      return launch_pair<kOutF32LseAllowed>(mx, mw, my, M, N, K, relu, s, reinterpret_cast<float2*>(lse_part), aff,
                                            AllowedStores{allow_bits, y_f32, ldy});
    if (aff.in_kernel_stats) {
      if (f32) return lse_part != nullptr
                          ? launch_pair<kOutF32Lse, true>(mx, mw, my, M, N, K, relu, s, reinterpret_cast<float2*>(lse_part), aff)
                          : launch_pair<kOutF32, true>(mx, mw, my, M, N, K, relu, s, nullptr, aff);
      return launch_pair<kOutBf16, true>(mx, mw, my, M, N, K, relu, s, nullptr, aff);
    }
    if (!f32) return add_into_bf16 ? launch_pair<kOutBf16Add>(mx, mw, my, M, N, K, relu, s)
                                   : launch_pair<kOutBf16>(mx, mw, my, M, N, K, relu, s, nullptr, aff);
    if (lse_part != nullptr)
      return launch_pair<kOutF32Lse>(mx, mw, my, M, N, K, relu, s, reinterpret_cast<float2*>(lse_part), aff);
    if (aliased) return launch_pair<kOutF32Add>(mx, mw, my, M, N, K, relu, s);
    return launch_pair<kOutF32>(mx, mw, my, M, N, K, relu, s, nullptr, aff);
  }
  CUtensorMap mx, mw;
  // a grid that leaves most SMs idle is latency-bound: narrower tiles (more CTAs) and the whole K in flight
  const bool latency_form = (int64_t)((M + kGemmBM - 1) / kGemmBM) * ((N + 127) / 128) < 74;
  const int BN = (N >= 128 && !latency_form) ? 128 : (latency_form ? 32 : 64);
  {
    const uint64_t dims[2] = {(uint64_t)K, (uint64_t)M}, str[1] = {(uint64_t)ldx};
    const uint32_t box[2] = {(uint32_t)kGemmBK, (uint32_t)kGemmBM};
    if (!tc::make_tmap_bf16(&mx, x, 2, dims, str, box)) return GRACE_CUDA_ERROR;
  }
  {
    const uint64_t dims[2] = {(uint64_t)K, (uint64_t)N}, str[1] = {(uint64_t)ldw};
    const uint32_t box[2] = {(uint32_t)kGemmBK, (uint32_t)BN};
    if (!tc::make_tmap_bf16(&mw, w, 2, dims, str, box)) return GRACE_CUDA_ERROR;
  }
  GemmParams p;
  p.y_bf16 = y_bf16; p.y_f32 = y_f32; p.residual = residual; p.residual_bf16 = add_into_bf16 ? y_bf16 : nullptr;
  p.aff_row = aff.row; p.aff_cs = aff.cs; p.aff_cb = aff.cb;
  p.ldy = ldy; p.M = M; p.N = N; p.K = K; p.relu = relu;
  if (BN == 128) return launch_linear<128, 3>(mx, mw, p, s);
  return latency_form ? launch_linear<32, 8>(mx, mw, p, s) : launch_linear<64, 3>(mx, mw, p, s);
}

extern "C" grace_status_t grace_linear(const uint16_t* x, int64_t ldx, const uint16_t* w, int64_t ldw,
                                       uint16_t* y_bf16, float* y_f32, int64_t ldy, const float* residual,
                                       int M, int N, int K, int relu, void* stream) {
  return linear_impl(x, ldx, w, ldw, y_bf16, y_f32, ldy, residual, false, M, N, K, relu, stream);
}

extern "C" grace_status_t grace_linear_f32_lse(const uint16_t* x, int64_t ldx, const uint16_t* w, int64_t ldw,
                                               float* y_f32, int64_t ldy, float* lse_part, int M, int N, int K,
                                               void* stream) {
  if (!lse_part || (reinterpret_cast<uintptr_t>(lse_part) & 7)) return GRACE_INVALID_ARG;
  return linear_impl(x, ldx, w, ldw, nullptr, y_f32, ldy, nullptr, false, M, N, K, 0, stream, lse_part);
}

extern "C" grace_status_t grace_linear_folded_ln(const uint16_t* x, int64_t ldx, const uint16_t* w, int64_t ldw,
                                                 const float* row_affine, const float* col_sum, const float* col_bias,
                                                 uint16_t* y_bf16, float* y_f32, int64_t ldy, float* lse_part,
                                                 int M, int N, int K, int relu, void* stream) {
  if (!row_affine || !col_bias || (reinterpret_cast<uintptr_t>(row_affine) & 7) ||
      !grace_aligned16(col_sum) || !grace_aligned16(col_bias))
    return GRACE_INVALID_ARG;
  if (lse_part != nullptr && (reinterpret_cast<uintptr_t>(lse_part) & 7)) return GRACE_INVALID_ARG;
  grace::Affine aff = {reinterpret_cast<const float2*>(row_affine), col_sum, col_bias};
  return linear_impl(x, ldx, w, ldw, y_bf16, y_f32, ldy, nullptr, false, M, N, K, relu, stream, lse_part, aff);
}

extern "C" grace_status_t grace_linear_layer_norm(const uint16_t* x, int64_t ldx, const uint16_t* w, int64_t ldw,
                                                  float eps, float* row_affine, const float* col_sum,
                                                  const float* col_bias, uint16_t* y_bf16, float* y_f32, int64_t ldy,
                                                  float* lse_part, int M, int N, int K, int relu, void* stream) {
  if (!row_affine || !col_bias || (reinterpret_cast<uintptr_t>(row_affine) & 7) ||
      !grace_aligned16(col_sum) || !grace_aligned16(col_bias))
    return GRACE_INVALID_ARG;
  if (lse_part != nullptr && (reinterpret_cast<uintptr_t>(lse_part) & 7)) return GRACE_INVALID_ARG;
  if (M <= 0 || N <= 0 || K <= 0 || ldx != K) return GRACE_INVALID_ARG;     // the LayerNorm is over the whole row of x
  grace::Affine aff = {reinterpret_cast<const float2*>(row_affine), col_sum, col_bias};
  // The statistics come out of the GEMM's own operand tiles where the CTA-pair kernel runs, the rows are centred
  // (no col_sum) and the output is at most two tiles wide; otherwise the statistics kernel runs first, into
  // row_affine.  Every n-tile forms the statistics of its rows again, and the shared-memory reads that takes
  // (16 KB per k-block on top of the 32 KB the tensor cores read and the 32 KB TMA writes) slow the main loop by a
  // fifth: measured at 65536 x 512 -> N, one kernel against two: N = 512: 36 us against 43; N = 1536: 99 against
  // 95; N = 2048: 130 against 122.
  const bool pair_kernel = (M >= 1024 && N >= 256);
  // (not for a logits GEMM with log-sum-exp partials: grace_linear_logits_allowed takes its statistics from the
  // statistics kernel, and the two forms of a decode step are to agree bit for bit)
  if (pair_kernel && col_sum == nullptr && N <= 512 && lse_part == nullptr) {
    aff.eps = eps;
    aff.in_kernel_stats = true;
  } else {
    const grace_status_t st = grace_row_stats_bf16(x, M, K, eps, row_affine, stream);
    if (st != GRACE_OK) return st;
  }
  return linear_impl(x, ldx, w, ldw, y_bf16, y_f32, ldy, nullptr, false, M, N, K, relu, stream, lse_part, aff);
}

extern "C" grace_status_t grace_linear_logits_allowed(const uint16_t* x, int64_t ldx, const uint16_t* w, int64_t ldw,
                                                      float eps, float* row_affine, const float* col_sum,
                                                      const float* col_bias, const uint64_t* allow_bits, float* y_f32,
                                                      int64_t ldy, float* lse_part, int M, int N, int K, void* stream) {
  if (!allow_bits || !y_f32 || !lse_part || (reinterpret_cast<uintptr_t>(lse_part) & 7)) return GRACE_INVALID_ARG;
  if (M < 1024 || N < 256 || (N % 256)) return GRACE_UNSUPPORTED_SHAPE;
  grace::Affine aff = {nullptr, nullptr, nullptr};
  if (row_affine != nullptr) {                              // a LayerNorm in front: statistics first, folded epilogue
    if (!col_bias || (reinterpret_cast<uintptr_t>(row_affine) & 7) || !grace_aligned16(col_sum) ||
        !grace_aligned16(col_bias) || ldx != K)
      return GRACE_INVALID_ARG;
    if (eps >= 0.f) {                                       // eps < 0: the caller has run grace_row_stats_bf16 into row_affine
      const grace_status_t st = grace_row_stats_bf16(x, M, K, eps, row_affine, stream);
      if (st != GRACE_OK) return st;
    }
    aff = grace::Affine{reinterpret_cast<const float2*>(row_affine), col_sum, col_bias};
  }
  return linear_impl(x, ldx, w, ldw, nullptr, y_f32, ldy, nullptr, false, M, N, K, 0, stream, lse_part, aff, allow_bits);
}

extern "C" grace_status_t grace_linear_add_bf16(const uint16_t* x, int64_t ldx, const uint16_t* w, int64_t ldw,
                                                uint16_t* y_inout, int64_t ldy, int M, int N, int K, void* stream) {
  return linear_impl(x, ldx, w, ldw, y_inout, nullptr, ldy, nullptr, true, M, N, K, 0, stream);
}

// ---------------------------------------------------------------------------------------------
// Bounded waits, checked without hanging anything: a one-block kernel waits on a barrier that
// nothing ever arrives on, with a limit of 64 parked polls (about a millisecond).
// ---------------------------------------------------------------------------------------------
namespace grace {
__global__ void bounded_wait_selftest_kernel(int* result) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    tc::mbar_init(&bar, 1);
    abort_flag = 0;
    tc::fence_mbar_init();
    const bool arrived = tc::mbar_wait<64>(&bar, 0, &abort_flag);
    *result = arrived ? 1 : (abort_flag ? 2 : 3);          // 2: gave up and raised the CTA's abort flag
  }
}
int linear_tc_timeouts() { return tc::tc_timeouts_read_and_clear(); }
static __device__ int g_selftest_result;
}  // namespace grace

extern "C" grace_status_t grace_selftest_bounded_wait(void* stream) {
  int* d_result = nullptr;
  GRACE_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&d_result), grace::g_selftest_result));
  grace::bounded_wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(d_result);
  GRACE_LAUNCH_CHECK();
  GRACE_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
  int h = 0;
  GRACE_CUDA_TRY(cudaMemcpy(&h, d_result, sizeof(int), cudaMemcpyDeviceToHost));
  return h == 2 ? GRACE_TIMEOUT : GRACE_CUDA_ERROR;
}
