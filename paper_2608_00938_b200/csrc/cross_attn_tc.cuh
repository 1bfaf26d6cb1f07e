// Cross-attention on tcgen05 tensor cores (Section 5.1: beams of a request are the M dimension of
// a dense contraction against that request's shared K/V).  Written for head size 64 or 128; the library
// uses it for head size 128 (head size 64 runs the four-stream kernel of cross_attn_ms.cuh).
//
// A work item is 128 query rows of one (request, head); its encoder positions are streamed in
// blocks of 128:
//   S   = Q K_blk^T        tcgen05.mma, A = Q (shared, K-major), B = K_blk (shared, K-major),
//                          fp32 S[128 x 128] in TMEM
//   P   = exp2(S*c - max)  softmax threads: TMEM lane = query row; two threads per row, half of the block's
//                          columns each (256 threads); P goes to its own TMEM columns as packed bf16
//   O  += P V_blk          tcgen05.mma, A = P (TMEM), B = V_blk (shared, read MN-major, so V is
//                          used as stored: no transpose anywhere); O stays in TMEM for the whole
//                          row tile and is rescaled lazily, only when a row maximum grows by > 2^8
// K and V blocks arrive by TMA through two separate two-slot rings; Q, K and V are addressed with 4-D tensor
// maps over the caller's strides, so the beam-major Q / O layout is never permuted (the view /
// permute / reshape chain of Section 5.1 costs nothing).  Ragged M and T are zero-filled by TMA
// and masked in the softmax.  Warp roles: softmax + epilogue warps first, then the TMA producer warp, then
// the MMA issuer warp.
// The kernel is persistent (each CTA loops over work items; Q is double-buffered), one CTA per SM with all
// 512 TMEM columns: S (128), O twice (by item parity) and P twice (by block parity).  The softmax threads
// therefore never wait for P V: they hand P of a block over and go on to the next block (whose S the tensor
// core produced under their exponentials), and an item's output is read from TMEM and stored one block later.
// A 128-wide tile is held as two 64-wide halves (the 128-byte swizzle spans 64 bf16), each with its own TMA
// box and its own MMA k-steps (Q, K) or output-column half (V).
#pragma once
#include "common.cuh"
#include "tc.cuh"

namespace grace {

constexpr int kCaBM = 128;        // query rows per work item
constexpr int kCaBN = 128;        // encoder positions per block
constexpr int kCaStages = 2;
constexpr int kCaHalfBytes = 128 * 64 * 2;                       // 16 KB: 128 rows x 64 bf16, one swizzle span wide
// TPR = softmax threads per query row: 2 (eight softmax warps, each thread half of a block's columns) or
// 1 (four softmax warps, a thread owns the whole row: no exchange between threads, half as many trips
// through the TMEM load / barrier / TMEM store sequence per exponential; 168 registers).  Head size 64
// runs TPR = 1 (4 % faster at 32 x 2048 x 1024); head size 128 keeps TPR = 2 for its wider output rows.
constexpr int kCaBarBytes = 256;
template <int DH> struct CaCfg {
  static constexpr int kHalves = DH / 64;
  static constexpr int kTileBytes = kCaHalfBytes * kHalves;      // Q, K_blk or V_blk
  static constexpr int kSmemBytes = kTileBytes * (2 + 2 * kCaStages) + 1024 + kCaBarBytes + 2 * 2 * 128 * 4 + 2 * 2 * 128 * 4;
  static constexpr uint32_t kTmemCols = 512;                     // S: 0..127, O: 2 x DH (by item parity), P: 2 x 64 (by block parity)
  static constexpr int kCtasPerSm = 1;
};

struct CrossTcParams {
  uint16_t* out;
  float* lse;
  int64_t out_row_stride;
  int B, M, H, T;
  int tiles_m, total_items;
  float scale_log2;             // scale * log2(e)
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float m;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(m) : "f"(a), "f"(b), "f"(c));
  return m;
}

// Persistent kernel: a flat grid of two CTAs per SM; CTA g takes the work items g, g + gridDim.x,
// ...  An item is one (request, head, 128-row tile); consecutive items are the tiles of the same
// (request, head), so the CTAs running at the same time read the same K/V from L2.
template <int DH, int TPR>
__global__ void __launch_bounds__((4 * TPR + 2) * 32, CaCfg<DH>::kCtasPerSm)
cross_attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                     const __grid_constant__ CUtensorMap map_v, const CrossTcParams p) {
  constexpr int kCaSoftmaxWarps = 4 * TPR;
  constexpr int kCols = kCaBN / TPR;                       // score columns per softmax thread and block
  constexpr int kCaTileBytes = CaCfg<DH>::kTileBytes, kHalves = CaCfg<DH>::kHalves;
  constexpr uint32_t kCaTmemCols = CaCfg<DH>::kTmemCols;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* q_tiles = tiles;                                      // two Q buffers
  uint8_t* kv_tiles = tiles + 2 * kCaTileBytes;                  // stage s: K at 2s, V at 2s+1
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + kCaTileBytes * (2 + 2 * kCaStages));
  uint64_t* q_full = bars;                    // [2]
  uint64_t* q_empty = bars + 2;               // [2]
  uint64_t* k_full = bars + 4;                // [stages]  K and V have separate rings: a K slot is
  uint64_t* k_empty = k_full + kCaStages;     // [stages]  free once S of its block has run, a V
  uint64_t* v_full = k_empty + kCaStages;     // [stages]  slot only after P V of its block
  uint64_t* v_empty = v_full + kCaStages;     // [stages]
  uint64_t* s_full = v_empty + kCaStages;
  uint64_t* p_full = s_full + 1;
  uint64_t* o_full = p_full + 1;              // [2] by block parity: P V of the block is complete
  uint64_t* s_free = o_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_free + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* half_max = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(bars) + kCaBarBytes);   // [2][2][128]
  float* half_sum = half_max + 2 * 2 * 128;                                                     // [2][128]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int NB = (p.T + kCaBN - 1) / kCaBN;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) { tc::mbar_init(q_full + i, 1); tc::mbar_init(q_empty + i, 1); }
    for (int s = 0; s < kCaStages; ++s) {
      tc::mbar_init(k_full + s, 1); tc::mbar_init(k_empty + s, 1);
      tc::mbar_init(v_full + s, 1); tc::mbar_init(v_empty + s, 1);
    }
    tc::mbar_init(s_full, 1);
    tc::mbar_init(p_full, kCaSoftmaxWarps);    // one arrival per softmax warp
    tc::mbar_init(o_full, 1);
    tc::mbar_init(o_full + 1, 1);
    tc::mbar_init(s_free, kCaSoftmaxWarps);
    *abort_flag = 0;
    tc::fence_mbar_init();
  }
  if (warp == kCaSoftmaxWarps) tc::tmem_alloc(tmem_slot, kCaTmemCols);
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();                                  // barrier set-up and TMEM allocation overlapped the previous kernel's tail
  pdl_trigger();
  const uint32_t tmem_s = tmem_base;           // S fp32, 128 columns
  // O of an item lives in one of two accumulators (item parity) and P of a block in one of two column sets (block
  // parity), so the softmax threads hand P(g) over and go straight on to block g + 1 (whose S is already there)
  // while the tensor core runs P V of block g; an item's output is read and stored one block later, when its last
  // P V has long finished.  With one K/V block per item (128 encoder positions) that takes the wait for P V and
  // most of the output path out of the per-item chain.
  static_assert(128 + 2 * DH + 2 * 64 <= 512, "TMEM columns");
  const uint32_t tmem_o = tmem_base + 128;             // O fp32, 2 x DH columns
  const uint32_t tmem_p = tmem_base + 128 + 2 * DH;    // P bf16 pairs, 2 x 64 columns

  if (warp == kCaSoftmaxWarps) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      tc::tma_prefetch_desc(&map_q); tc::tma_prefetch_desc(&map_k); tc::tma_prefetch_desc(&map_v);
      // One thread feeds three queues (Q per item, K and V per block).  K of block g+2 can be
      // requested as soon as S of block g has run, long before the V slot of block g frees, so the
      // thread polls: whichever slot is free next gets its load, neither queue blocks the other.
      const int my_items = (p.total_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
      const int total_blocks = my_items * NB;
      int gk = 0, gv = 0;                                    // next K block, next V block (global indices)
      int idle = 0;
      while ((gk < total_blocks || gv < total_blocks) && !*abort_flag) {
        bool progressed = false;
        if (gk < total_blocks) {
          const int li = gk / NB, j = gk - li * NB, s = gk % kCaStages;
          const int item = (int)blockIdx.x + li * (int)gridDim.x;
          const int bh = item / p.tiles_m, h = bh % p.H, b = bh / p.H;
          const bool need_q = (j == 0);
          const int qb = li & 1;
          if (tc::mbar_try_wait_now(k_empty + s, ((gk / kCaStages) & 1) ^ 1) &&
              (!need_q || tc::mbar_try_wait_now(q_empty + qb, ((li >> 1) & 1) ^ 1))) {
            if (need_q) {
              tc::mbar_expect_tx(q_full + qb, kCaTileBytes);
#pragma unroll
              for (int hf = 0; hf < kHalves; ++hf)
                tc::tma_load_4d(q_tiles + qb * kCaTileBytes + hf * kCaHalfBytes, &map_q, q_full + qb, 64 * hf, h,
                                (item % p.tiles_m) * kCaBM, b);
            }
            tc::mbar_expect_tx(k_full + s, kCaTileBytes);
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf)
              tc::tma_load_4d(kv_tiles + (2 * s) * kCaTileBytes + hf * kCaHalfBytes, &map_k, k_full + s, 64 * hf, j * kCaBN, h, b);
            ++gk;
            progressed = true;
          }
        }
        if (gv < total_blocks && gv < gk) {
          const int li = gv / NB, j = gv - li * NB, s = gv % kCaStages;
          const int item = (int)blockIdx.x + li * (int)gridDim.x;
          const int bh = item / p.tiles_m, h = bh % p.H, b = bh / p.H;
          if (tc::mbar_try_wait_now(v_empty + s, ((gv / kCaStages) & 1) ^ 1)) {
            tc::mbar_expect_tx(v_full + s, kCaTileBytes);
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf)
              tc::tma_load_4d(kv_tiles + (2 * s + 1) * kCaTileBytes + hf * kCaHalfBytes, &map_v, v_full + s, 64 * hf, j * kCaBN, h, b);
            ++gv;
            progressed = true;
          }
        }
        if (progressed) {
          idle = 0;
        } else {
          __nanosleep(512);                                 // polling costs issue slots the softmax warps of this scheduler need
          if (++idle > (1 << 24)) {                          // bounded: about a second of nothing to do
            if (*abort_flag == 0) atomicAdd(&tc::g_tc_timeouts, 1);
            *abort_flag = 1;
          }
        }
      }
    }
  } else if (warp == kCaSoftmaxWarps + 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc_s = tc::idesc_bf16(kCaBM, kCaBN, 0);     // Q K^T : B K-major
      constexpr uint32_t idesc_o = tc::idesc_bf16(kCaBM, 64, 1);        // P V   : B MN-major, 64 output columns at a time
      const int my_items = (p.total_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
      const int total_blocks = my_items * NB;
      // Every operand descriptor is fixed by (Q buffer, ring slot, k-step): build them once.  The
      // issuing thread shares its scheduler with busy softmax warps, so each instruction it does not
      // execute per block shortens the hand-off to the tensor core.
      // k-step k of Q or K: 16 of the DH columns = 32 bytes inside the 64-wide half (k / 4)
      uint64_t q_desc[2][DH / 16], k_desc[kCaStages][DH / 16], v_desc[kCaStages][kHalves][kCaBN / 16];
#pragma unroll
      for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int k = 0; k < DH / 16; ++k)
          q_desc[i][k] = tc::smem_desc_sw128(tc::smem_addr(q_tiles + i * kCaTileBytes) + (k / 4) * kCaHalfBytes + 32 * (k % 4), 16, 1024);
#pragma unroll
      for (int st = 0; st < kCaStages; ++st) {
#pragma unroll
        for (int k = 0; k < DH / 16; ++k)
          k_desc[st][k] = tc::smem_desc_sw128(tc::smem_addr(kv_tiles + (2 * st) * kCaTileBytes) + (k / 4) * kCaHalfBytes + 32 * (k % 4), 16, 1024);
#pragma unroll
        for (int hf = 0; hf < kHalves; ++hf)
#pragma unroll
          for (int k = 0; k < kCaBN / 16; ++k)
            v_desc[st][hf][k] = tc::smem_desc_sw128(tc::smem_addr(kv_tiles + (2 * st + 1) * kCaTileBytes) + hf * kCaHalfBytes + 2048 * k, 1024, 1024);
      }
      // S of global block g: Q buffer of its item, K of ring slot g % stages
      auto issue_s = [&](int g, int j, int li) -> bool {
        const int qb = li & 1, s = g % kCaStages;
        if (j == 0 && !tc::mbar_wait(q_full + qb, (li >> 1) & 1, abort_flag)) return false;
        if (!tc::mbar_wait(k_full + s, (g / kCaStages) & 1, abort_flag)) return false;
        tc::tc_fence_after();
        if (qb == 0) {
          if (s == 0) {
#pragma unroll
            for (int k = 0; k < DH / 16; ++k) tc::mma_ss(tmem_s, q_desc[0][k], k_desc[0][k], idesc_s, k ? 1u : 0u);
          } else {
#pragma unroll
            for (int k = 0; k < DH / 16; ++k) tc::mma_ss(tmem_s, q_desc[0][k], k_desc[1][k], idesc_s, k ? 1u : 0u);
          }
        } else {
          if (s == 0) {
#pragma unroll
            for (int k = 0; k < DH / 16; ++k) tc::mma_ss(tmem_s, q_desc[1][k], k_desc[0][k], idesc_s, k ? 1u : 0u);
          } else {
#pragma unroll
            for (int k = 0; k < DH / 16; ++k) tc::mma_ss(tmem_s, q_desc[1][k], k_desc[1][k], idesc_s, k ? 1u : 0u);
          }
        }
        tc::mma_commit(s_full);
        tc::mma_commit(k_empty + s);                         // K of block g is consumed
        if (j == NB - 1) tc::mma_commit(q_empty + qb);       // last use of this item's Q tile
        return true;
      };
      static_assert(kCaStages == 2, "descriptor selection below is written for two ring slots");
      bool ok = total_blocks > 0 && issue_s(0, 0, 0);
      int j = 0, li = 0;                                     // block inside the item, local item index
      for (int g = 0; ok && g < total_blocks; ++g) {
        const int s = g & 1;
        int j1 = j + 1, li1 = li;
        if (j1 == NB) { j1 = 0; ++li1; }
        // s_free(g): every softmax thread holds its scores of block g in registers, so the S
        // columns can be overwritten: S of block g+1 (possibly the next item's first block) runs
        // on the tensor core while the exponentials of block g are computed.
        if (!tc::mbar_wait(s_free, g & 1, abort_flag)) break;
        if (g + 1 < total_blocks && !issue_s(g + 1, j1, li1)) break;
        // p_full(g): P of block g is in its TMEM columns (and, on an item's first block, the
        // previous item's epilogue has read O).
        if (!tc::mbar_wait(p_full, g & 1, abort_flag)) break;
        if (!tc::mbar_wait(v_full + s, (g >> 1) & 1, abort_flag)) break;
        tc::tc_fence_after();
        const uint32_t o_acc = tmem_o + (uint32_t)((li & 1) * DH), p_cols = tmem_p + (uint32_t)((g & 1) * 64);
        if (s == 0) {
#pragma unroll
          for (int hf = 0; hf < kHalves; ++hf)
#pragma unroll
            for (int k = 0; k < kCaBN / 16; ++k)
              tc::mma_ts(o_acc + 64 * hf, p_cols + 8 * k, v_desc[0][hf][k], idesc_o, (j | k) ? 1u : 0u);
        } else {
#pragma unroll
          for (int hf = 0; hf < kHalves; ++hf)
#pragma unroll
            for (int k = 0; k < kCaBN / 16; ++k)
              tc::mma_ts(o_acc + 64 * hf, p_cols + 8 * k, v_desc[1][hf][k], idesc_o, (j | k) ? 1u : 0u);
        }
        tc::mma_commit(v_empty + s);                         // V of block g is consumed
        tc::mma_commit(o_full + (g & 1));                    // O includes block g
        j = j1; li = li1;
      }
    }
  } else {
    // ---------------- softmax + epilogue ----------------
    // Warps w and w+4 share the TMEM lanes (= query rows) 32*(w&3)..+31; each takes one half of the
    // 128 score columns and one half of the DH output columns of those rows.  O stays in TMEM and
    // accumulates across blocks; it is rescaled only when a row's maximum grows by more than 2^8
    // (probabilities may then reach 256, which bf16 and the fp32 sums hold without loss).
    const int quarter = warp & 3, half = warp >> 2;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const int col_base = kCols * half;
    constexpr int kOutCols = DH / TPR;                     // output columns per thread
    bool ok = true;
    int g = 0, n_done = 0, li = 0;
    // the item whose output is still to be read from TMEM and stored (after the next block's P hand-over)
    int pend_item = -1, pend_g = 0, pend_li = 0;
    float pend_m = 0.f, pend_l = 0.f;
    // wait for P V of global block gb (completion gb >> 1 of the barrier of its parity)
    auto wait_pv = [&](int gb) -> bool {
      bool w = tc::mbar_wait(o_full + (gb & 1), (gb >> 1) & 1, abort_flag);
      return __all_sync(kFullMask, w);
    };
    auto store_item = [&](int item_e, int g_last, int li_e, float m_e, float l_e) -> bool {
      const int tile = item_e % p.tiles_m, bh = item_e / p.tiles_m;
      const int h = bh % p.H, b = bh / p.H;
      if (!wait_pv(g_last)) return false;
      tc::tc_fence_after();
      const uint32_t o_acc = tmem_o + (uint32_t)((li_e & 1) * DH);
      uint32_t o[kOutCols];
#pragma unroll
      for (int c = 0; c < kOutCols; c += 32)
        tc::tmem_ld32(o_acc + lane_addr + kOutCols * half + c, *reinterpret_cast<uint32_t(*)[32]>(&o[c]));
      tc::tmem_ld_wait();
      float l_tot = l_e;
      if (TPR == 2) {
        float* hs = half_sum + (n_done & 1) * 256;            // double-buffered by item parity
        hs[half * 128 + row] = l_e;
        tc::named_bar_sync(2 + quarter, 64);
        l_tot += hs[(half ^ 1) * 128 + row];
      }
      ++n_done;
      const int m = tile * kCaBM + row;
      if (m < p.M) {
        const float inv = 1.f / l_tot;
        const int64_t r_out = (int64_t)b * p.M + m;
        uint4* dst = reinterpret_cast<uint4*>(p.out + r_out * p.out_row_stride + h * DH + kOutCols * half);
        auto piece = [&](int i) {
          return make_uint4(
              pack_bf16x2(__uint_as_float(o[8 * i]) * inv, __uint_as_float(o[8 * i + 1]) * inv),
              pack_bf16x2(__uint_as_float(o[8 * i + 2]) * inv, __uint_as_float(o[8 * i + 3]) * inv),
              pack_bf16x2(__uint_as_float(o[8 * i + 4]) * inv, __uint_as_float(o[8 * i + 5]) * inv),
              pack_bf16x2(__uint_as_float(o[8 * i + 6]) * inv, __uint_as_float(o[8 * i + 7]) * inv));
        };
        // a thread owns a row: its stores are pieces at a row stride, so whole 32-byte sectors where the
        // output's alignment allows (half the store transactions of 16-byte pieces)
        if ((reinterpret_cast<uintptr_t>(dst) & 31) == 0) {
#pragma unroll
          for (int i = 0; i < kOutCols / 8; i += 2) st_global_32B(dst + i, piece(i), piece(i + 1));
        } else {
#pragma unroll
          for (int i = 0; i < kOutCols / 8; ++i) dst[i] = piece(i);
        }
        if (p.lse != nullptr && half == 0) p.lse[r_out * p.H + h] = (m_e + log2f(l_tot)) * 0.6931471805599453f;
      }
      // the accumulator is free for the item after next: its first P V is issued only after these threads have
      // arrived on p_full for that item's first block, which comes after this read in program order
      tc::tc_fence_before();
      return true;
    };
    for (int item = blockIdx.x; ok && item < p.total_items; item += gridDim.x, ++li) {
      const uint32_t o_acc = tmem_o + (uint32_t)((li & 1) * DH);
      float m_run = -INFINITY, l_run = 0.f;
      for (int j = 0; j < NB; ++j, ++g) {
        ok = ok && tc::mbar_wait(s_full, g & 1, abort_flag);
        ok = __all_sync(kFullMask, ok);
        if (!ok) break;
        tc::tc_fence_after();
        uint32_t r[kCols];
        {
#pragma unroll
          for (int c = 0; c < kCols; c += 32)
            tc::tmem_ld32(tmem_s + lane_addr + col_base + c, *reinterpret_cast<uint32_t(*)[32]>(&r[c]));
          tc::tmem_ld_wait();
        }
        tc::tc_fence_before();
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(s_free);              // the scores now live in registers
        const int valid = min(kCaBN, p.T - j * kCaBN) - col_base;   // this thread's columns that exist
        if (valid < kCols) {
#pragma unroll
          for (int i = 0; i < kCols; ++i)
            if (i >= valid) r[i] = 0xff800000u;                     // -inf: no weight, no influence on the max
        }
        // four independent chains instead of one 32-deep one
        float mx0 = max3(__uint_as_float(r[0]), __uint_as_float(r[1]), __uint_as_float(r[2]));
        float mx1 = max3(__uint_as_float(r[3]), __uint_as_float(r[4]), __uint_as_float(r[5]));
        float mx2 = max3(__uint_as_float(r[6]), __uint_as_float(r[7]), __uint_as_float(r[8]));
        float mx3 = max3(__uint_as_float(r[9]), __uint_as_float(r[10]), __uint_as_float(r[11]));
#pragma unroll
        for (int i = 12; i + 7 < kCols; i += 8) {
          mx0 = max3(mx0, __uint_as_float(r[i]), __uint_as_float(r[i + 1]));
          mx1 = max3(mx1, __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
          mx2 = max3(mx2, __uint_as_float(r[i + 4]), __uint_as_float(r[i + 5]));
          mx3 = max3(mx3, __uint_as_float(r[i + 6]), __uint_as_float(r[i + 7]));
        }
        mx0 = max3(mx0, __uint_as_float(r[kCols - 4]), __uint_as_float(r[kCols - 3]));
        mx1 = max3(mx1, __uint_as_float(r[kCols - 2]), __uint_as_float(r[kCols - 1]));
        float mx = fmaxf(max3(mx0, mx1, mx2), mx3);
        if (TPR == 2) {
          float* hm = half_max + (g & 1) * 256;
          hm[half * 128 + row] = mx;
          tc::named_bar_sync(2 + quarter, 64);                // the two warps of this row quarter
          mx = fmaxf(mx, hm[(half ^ 1) * 128 + row]);
        }
        const float m_blk = mx * p.scale_log2;
        const bool grow = m_blk > m_run + 8.0f;               // always true on an item's first block
        const float m_new = grow ? m_blk : m_run;
        const float alpha = grow ? ex2(m_run - m_new) : 1.0f; // 0 on the first block
        m_run = m_new;
        // probabilities -> packed bf16 in the P columns; row sum in four independent accumulators
        const float neg_m = -m_new;
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
        for (int i = 0; i < kCols / 4; ++i) {
          const float e0 = ex2(fmaf(__uint_as_float(r[4 * i]), p.scale_log2, neg_m));
          const float e1 = ex2(fmaf(__uint_as_float(r[4 * i + 1]), p.scale_log2, neg_m));
          const float e2 = ex2(fmaf(__uint_as_float(r[4 * i + 2]), p.scale_log2, neg_m));
          const float e3 = ex2(fmaf(__uint_as_float(r[4 * i + 3]), p.scale_log2, neg_m));
          s0 += e0; s1 += e1; s2 += e2; s3 += e3;
          r[2 * i] = pack_bf16x2(e0, e1);
          r[2 * i + 1] = pack_bf16x2(e2, e3);
        }
        l_run = fmaf(l_run, alpha, (s0 + s1) + (s2 + s3));
        if (g >= 2) {
          // the P columns of this parity were read by P V of block g - 2: long finished, but it must be
          ok = wait_pv(g - 2);
          if (!ok) break;
          tc::tc_fence_after();
        }
        {
#pragma unroll
          for (int c = 0; c < kCols / 2; c += 16)
            tc::tmem_st16(tmem_p + (uint32_t)((g & 1) * 64) + lane_addr + (kCols / 2) * half + c,
                          *reinterpret_cast<uint32_t(*)[16]>(&r[c]));
        }
        if (j > 0 && __any_sync(kFullMask, grow)) {           // rare after the first blocks
          // O changes under the tensor core only here: P V of block g - 1 (the same item) must be complete
          ok = wait_pv(g - 1);
          if (!ok) break;
          tc::tc_fence_after();
#pragma unroll
          for (int c = 0; c < kOutCols; c += 32) {
            uint32_t o[32];
            tc::tmem_ld32(o_acc + lane_addr + kOutCols * half + c, o);
            tc::tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
            uint32_t (&o0)[16] = *reinterpret_cast<uint32_t(*)[16]>(&o[0]);
            uint32_t (&o1)[16] = *reinterpret_cast<uint32_t(*)[16]>(&o[16]);
            tc::tmem_st16(o_acc + lane_addr + kOutCols * half + c, o0);
            tc::tmem_st16(o_acc + lane_addr + kOutCols * half + c + 16, o1);
          }
        }
        tc::tmem_st_wait();
        tc::tc_fence_before();
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(p_full);
        // the previous item's output, now that this block is with the tensor core
        if (pend_item >= 0) {
          ok = store_item(pend_item, pend_g, pend_li, pend_m, pend_l);
          pend_item = -1;
          if (!ok) break;
        }
      }
      if (!ok) break;
      pend_item = item; pend_g = g - 1; pend_li = li; pend_m = m_run; pend_l = l_run;
    }
    if (ok && pend_item >= 0) store_item(pend_item, pend_g, pend_li, pend_m, pend_l);
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == kCaSoftmaxWarps) tc::tmem_dealloc(tmem_base, kCaTmemCols);
}

inline bool cross_attn_tc_supported(int B, int M, int H, int d_h, int T_ctx) {
  return d_h == 128 && H <= 65535 && B <= 65535 && T_ctx >= 1 && M >= 1;      // head size 64: cross_attn_ms.cuh
}

template <int DH, int TPR>
inline grace_status_t launch_cross_attn_tc_dh(const uint16_t* q, int64_t q_row_stride, const uint16_t* k,
                                              const uint16_t* v, int64_t kv_stride_b, int64_t kv_stride_h,
                                              int64_t kv_stride_t, uint16_t* out, int64_t out_row_stride, float* lse,
                                              int B, int M, int H, int T_ctx, float scale, cudaStream_t s) {
  constexpr int kCaSmemBytes = CaCfg<DH>::kSmemBytes;
  CUtensorMap mq, mk, mv;
  {
    const uint64_t dims[4] = {(uint64_t)DH, (uint64_t)H, (uint64_t)M, (uint64_t)B};
    const uint64_t str[3] = {(uint64_t)DH, (uint64_t)q_row_stride, (uint64_t)M * (uint64_t)q_row_stride};
    const uint32_t box[4] = {64u, 1u, (uint32_t)kCaBM, 1u};
    if (!tc::make_tmap_bf16(&mq, q, 4, dims, str, box)) return GRACE_CUDA_ERROR;
  }
  {
    const uint64_t dims[4] = {(uint64_t)DH, (uint64_t)T_ctx, (uint64_t)H, (uint64_t)B};
    const uint64_t str[3] = {(uint64_t)kv_stride_t, (uint64_t)kv_stride_h, (uint64_t)kv_stride_b};
    const uint32_t box[4] = {64u, (uint32_t)kCaBN, 1u, 1u};
    if (!tc::make_tmap_bf16(&mk, k, 4, dims, str, box)) return GRACE_CUDA_ERROR;
    if (!tc::make_tmap_bf16(&mv, v, 4, dims, str, box)) return GRACE_CUDA_ERROR;
  }
  static unsigned long long attr_set_devices = 0;
  static int n_sm_of[kMaxDevices] = {0};
  DeviceSetup su(&attr_set_devices);
  if (su) {
    GRACE_CUDA_TRY(cudaFuncSetAttribute(cross_attn_tc_kernel<DH, TPR>, cudaFuncAttributeMaxDynamicSharedMemorySize, kCaSmemBytes));
    GRACE_CUDA_TRY(cudaDeviceGetAttribute(&n_sm_of[su.dev], cudaDevAttrMultiProcessorCount, su.dev));
    su.done();
  }
  const int n_sm = n_sm_of[su.dev];
  CrossTcParams p;
  p.out = out; p.lse = lse; p.out_row_stride = out_row_stride; p.B = B; p.M = M; p.H = H; p.T = T_ctx;
  p.tiles_m = (M + kCaBM - 1) / kCaBM;
  const int64_t items = (int64_t)p.tiles_m * H * B;
  if (items > 0x7fffffff) return GRACE_UNSUPPORTED_SHAPE;
  p.total_items = (int)items;
  p.scale_log2 = scale * 1.4426950408889634f;
  const int ctas = CaCfg<DH>::kCtasPerSm * n_sm;
  const int grid = (int)(items < ctas ? items : ctas);
  launch_pdl(cross_attn_tc_kernel<DH, TPR>, dim3(grid), dim3((4 * TPR + 2) * 32), kCaSmemBytes, s, mq, mk, mv, p);
  GRACE_LAUNCH_CHECK();
  return GRACE_OK;
}

inline grace_status_t launch_cross_attn_tc(const uint16_t* q, int64_t q_row_stride, const uint16_t* k,
                                           const uint16_t* v, int64_t kv_stride_b, int64_t kv_stride_h,
                                           int64_t kv_stride_t, uint16_t* out, int64_t out_row_stride, float* lse,
                                           int B, int M, int H, int d_h, int T_ctx, float scale, cudaStream_t s) {
  (void)d_h;                                                // 128 (cross_attn_tc_supported)
  return launch_cross_attn_tc_dh<128, 2>(q, q_row_stride, k, v, kv_stride_b, kv_stride_h, kv_stride_t, out, out_row_stride,
                                        lse, B, M, H, T_ctx, scale, s);
}

}  // namespace grace
