// Cross-attention on tcgen05 tensor cores, head size 64: four independent softmax streams per SM
// (Section 5.1: the beams of a request are the M dimension of a dense contraction against that
// request's shared K/V).
//
// What sets the pace at head size 64 (measured on B200, see the profiles directory):
//   * a 128 x 128 score block costs 512 tensor-core clocks but 16384 exponentials; the special-function
//     unit takes one warp instruction per 8 clocks and scheduler (1024 clocks per block and SM), and a
//     single warp can issue an exponential only every ~14 clocks: several warps per scheduler have to
//     be in the exponentials at any time;
//   * every tcgen05.mma / tcgen05.commit costs 32-48 clocks to ISSUE, and issue is serialised over the
//     whole SM whichever warp it comes from: the instruction count per block matters, not only the
//     flops (score sub-blocks of 32 columns needed 36 instructions per block and were issue-bound);
//   * every hand-off between warps or to the tensor core (mbarrier arrive -> wake, commit -> wake)
//     costs 150-250 clocks.
// Hence this layout:
//   * one CTA per SM owns all 512 TMEM columns and runs four streams.  A stream is one 128-row
//     query tile of one (request, head) with 64 score columns (S, fp32; the packed bf16
//     probabilities P overwrite the first 32 of them) and 64 output columns (O, fp32) in TMEM, its
//     own Q tiles in shared memory and its own barriers;
//   * streams 0/1 are the two tiles of one 256-row item and share that item's K/V ring, streams
//     2/3 those of another item with a second ring: two independent halves, so a request needs
//     only 256 beams to fill an SM;
//   * the encoder positions are walked in blocks of 64.  Four softmax warps per stream (one per
//     TMEM lane quarter, one thread per query row: 16 warps, four per scheduler) turn S of a block
//     into P; a fifth warp per stream issues the stream's MMAs in the order
//         S(0);   O += P(u) V(u),  S(u + 1)   for u = 0, 1, ...
//     running on into the next item (S(u + 1) overwrites the columns P(u) was read from; the
//     in-order tensor pipe makes that safe).  A stream's chain  S -> softmax -> P -> P V, next S
//     runs under the other three streams' exponentials; nothing is exchanged between streams;
//   * K and V arrive by TMA in blocks of 64 positions through three-slot rings per half; Q tiles
//     are double-buffered per stream, so the next item's first scores are computed under the
//     current item's epilogue.  Q, K, V and the output are addressed with 4-D tensor maps over the
//     caller's strides: the beam-major Q / O layout is never permuted;
//   * the epilogue stages the bf16 output rows in the Q tile the item no longer needs and writes
//     them with a TMA store per warp (rows beyond M are clipped by the tensor map).
//
// Ragged M and T are zero-filled by TMA and masked in the softmax; `enc_len` (optional) gives a
// per-request number of valid encoder positions (0: the output rows are zero).  Every wait is
// bounded (tc::mbar_wait); a wait that gives up sets the CTA's abort flag, every role leaves its
// loops, TMEM is freed and the kernel returns.
#pragma once
#include "common.cuh"
#include "tc.cuh"

namespace grace {

constexpr int kMsBM = 128;                 // query rows per tile (stream)
constexpr int kMsBN = 64;                  // encoder positions per K / V block in shared memory
constexpr float kMsGrowLog2 = 16.0f;       // the running reference maximum moves only when exceeded by this much
constexpr int kMsDH = 64;
constexpr int kMsStages = 3;               // K/V ring slots per half; a slot holds K and V of one block
constexpr int kMsQBytes = kMsBM * kMsDH * 2;       // 16 KB
constexpr int kMsKVBytes = kMsBN * kMsDH * 2;      // 8 KB
constexpr int kMsSoftmaxWarps = 16;
constexpr int kMsThreads = (kMsSoftmaxWarps + 4) * 32;   // + one MMA issuer / TMA producer warp per stream
constexpr int kMsBarBytes = 1024;
constexpr int kMsSmemBytes = 1024 + 8 * kMsQBytes + 2 * kMsStages * 2 * kMsKVBytes + kMsBarBytes;

struct CrossMsParams {
  float* lse;
  const int32_t* enc_len;       // nullable: valid encoder positions per request (<= T)
  uint16_t* out;                // only for rows without any encoder position (written as zeros)
  int64_t out_row_stride;
  int B, M, H, T;
  int pairs_m, total_items;     // 256-row items per (request, head); items = B * H * pairs_m
  float scale_log2;             // scale * log2(e)
};

__device__ __forceinline__ float ms_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float ms_max3(float a, float b, float c) {
  float m;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(m) : "f"(a), "f"(b), "f"(c));
  return m;
}

// One 256-row item: request, head, first query row, encoder positions, blocks, live tiles.
struct MsItem { int b, h, row0, T, nb, ntiles; };
__device__ __forceinline__ MsItem ms_item(const CrossMsParams& p, int item) {
  MsItem it;
  const int bh = item / p.pairs_m;
  const int pair = item - bh * p.pairs_m;
  it.b = bh / p.H;
  it.h = bh - it.b * p.H;
  it.row0 = pair * 2 * kMsBM;
  int t = p.T;
  if (p.enc_len != nullptr) { const int e = __ldg(p.enc_len + it.b); t = e < 0 ? 0 : (e < t ? e : t); }
  it.T = t;
  it.nb = (t + kMsBN - 1) / kMsBN;
  it.ntiles = p.M - it.row0 > kMsBM ? 2 : 1;
  return it;
}

__global__ void __launch_bounds__(kMsThreads, 1)
cross_attn_ms_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                     const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_o,
                     const CrossMsParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* q_tiles = tiles;                                      // [stream][buffer] x 16 KB
  uint8_t* kv_tiles = tiles + 8 * kMsQBytes;                     // [half][slot] x (K 8 KB, V 8 KB)
  uint64_t* bars = reinterpret_cast<uint64_t*>(kv_tiles + 2 * kMsStages * 2 * kMsKVBytes);
  uint64_t* q_full = bars;                          // [4][2] per stream and buffer
  uint64_t* q_empty = q_full + 8;                   // [4][2]  four arrivals: the stream's softmax warps, after their output stores
  uint64_t* kv_full = q_empty + 8;                  // [2][kMsStages]
  uint64_t* kv_empty = kv_full + 2 * kMsStages;     //        two arrivals: both streams of the half
  uint64_t* s_full = kv_empty + 2 * kMsStages;      // [4] S of the stream's next block is in TMEM
  uint64_t* p_full = s_full + 4;                    // [4] the stream's four warps have stored P
  uint64_t* o_full = p_full + 4;                    // [4] the stream's last P V of the item is done
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_full + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 8; ++i) { tc::mbar_init(q_full + i, 1); tc::mbar_init(q_empty + i, 4); }
    for (int i = 0; i < 4; ++i) { tc::mbar_init(s_full + i, 1); tc::mbar_init(p_full + i, 4); tc::mbar_init(o_full + i, 1); }
    for (int i = 0; i < 2 * kMsStages; ++i) { tc::mbar_init(kv_full + i, 1); tc::mbar_init(kv_empty + i, 2); }
    *abort_flag = 0;
    tc::fence_mbar_init();
  }
  if (warp == kMsSoftmaxWarps) tc::tmem_alloc(tmem_slot, 512);
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();                                  // barrier set-up and TMEM allocation overlapped the previous kernel's tail
  pdl_trigger();
  // Half `hf` of CTA c works on the items 2 (c + k gridDim) + hf, k = 0, 1, ...: the two halves of a
  // CTA and neighbouring CTAs run neighbouring items, which share K/V in L2.
  const int item_step = 2 * (int)gridDim.x;

  if (warp >= kMsSoftmaxWarps) {
    // ---------------- MMA issuer and TMA producer, one warp per stream ----------------
    // The whole warp walks the loops and tests the barriers; one elected lane issues (warp-uniform
    // control flow keeps the descriptors in uniform registers).  MMA order per stream, across items:
    //     S(0);   O += P(u) V(u),  S(u + 1)   for u = 0, 1, ...
    // The warp also requests the stream's Q tiles and, for the first stream of a half, the half's
    // K/V blocks: whenever it has to wait it first looks for a free slot to fill (refill), so loads
    // run ahead of the MMAs without a polling warp of their own.
    const int s = warp - kMsSoftmaxWarps;
    const int hf = s >> 1, tile = s & 1;
    const uint32_t tmem_s = tmem_base + 64 * s;
    const uint32_t tmem_o = tmem_base + 256 + 64 * s;
    constexpr uint32_t idesc_s = tc::idesc_bf16(kMsBM, kMsBN, 0);     // Q K^T : B K-major, 64 score columns
    constexpr uint32_t idesc_o = tc::idesc_bf16(kMsBM, kMsDH, 1);     // P V   : B MN-major, 64 output columns
    // Operand descriptors differ only in their start address (bits 0..13, in 16-byte units).
    const uint64_t q_desc0 = tc::smem_desc_sw128(tc::smem_addr(q_tiles + 2 * s * kMsQBytes), 16, 1024);
    uint8_t* const kv_half = kv_tiles + hf * kMsStages * 2 * kMsKVBytes;
    const uint64_t k_desc0 = tc::smem_desc_sw128(tc::smem_addr(kv_half), 16, 1024);
    const uint64_t v_desc0 = tc::smem_desc_sw128(tc::smem_addr(kv_half + kMsKVBytes), 1024, 1024);
    uint64_t* const kvf = kv_full + hf * kMsStages;
    uint64_t* const kve = kv_empty + hf * kMsStages;
    bool ok = true;
    if (lane == 0) { tc::tma_prefetch_desc(&map_q); tc::tma_prefetch_desc(&map_k); tc::tma_prefetch_desc(&map_v); }

    // ---- loads ----
    int lq_item = 2 * (int)blockIdx.x + hf, lq_cnt = 0;           // Q: next item to look at; tiles requested
    int lk_item = lq_item, lk_j = 0, lk_cnt = 0;                  // K/V (first stream of the half only): item, block, blocks requested
    MsItem lk_it = lk_item < p.total_items ? ms_item(p, lk_item) : MsItem{0, 0, 0, 0, 0, 0};
    MsItem lq_it = lk_it;                                          // an item is decoded when a queue moves on to it
    auto refill = [&]() -> bool {
      bool progressed = false;
      if (lq_item < p.total_items) {
        const MsItem& it = lq_it;
        bool advance = tile >= it.ntiles || it.nb == 0;             // nothing to load for this stream
        if (!advance) {
          const int buf = 2 * s + (lq_cnt & 1);
          if (tc::mbar_try_wait_now(q_empty + buf, ((lq_cnt >> 1) & 1) ^ 1)) {
            if (tc::elect_one()) {
              tc::mbar_expect_tx(q_full + buf, kMsQBytes);
              tc::tma_load_4d(q_tiles + buf * kMsQBytes, &map_q, q_full + buf, 0, it.h, it.row0 + tile * kMsBM, it.b);
            }
            __syncwarp();
            ++lq_cnt;
            advance = true;
          }
        }
        if (advance) {
          lq_item += item_step; progressed = true;
          if (lq_item < p.total_items) lq_it = ms_item(p, lq_item);
        }
      }
      if (tile == 0 && lk_item < p.total_items) {
        if (lk_j >= lk_it.nb) {
          lk_item += item_step; lk_j = 0; progressed = true;
          if (lk_item < p.total_items) lk_it = ms_item(p, lk_item);
        } else {
          const int slot = lk_cnt % kMsStages;
          if (tc::mbar_try_wait_now(kve + slot, ((lk_cnt / kMsStages) & 1) ^ 1)) {
            if (tc::elect_one()) {
              uint8_t* dst = kv_half + slot * 2 * kMsKVBytes;
              tc::mbar_expect_tx(kvf + slot, 2 * kMsKVBytes);
              tc::tma_load_4d(dst, &map_k, kvf + slot, 0, lk_j * kMsBN, lk_it.h, lk_it.b);
              tc::tma_load_4d(dst + kMsKVBytes, &map_v, kvf + slot, 0, lk_j * kMsBN, lk_it.h, lk_it.b);
              if (lk_it.ntiles == 1) tc::mbar_arrive(kve + slot);     // the half's second stream has no rows in this item
            }
            __syncwarp();
            ++lk_cnt; ++lk_j;
            progressed = true;
          }
        }
      }
      return progressed;
    };
    // A wait that keeps the loads going: test, refill, and only then park for a short while.
    auto wait_refilling = [&](uint64_t* bar, uint32_t parity) {
      int polls = 0;
      while (ok && !tc::mbar_try_wait_now(bar, parity)) {
        if (refill()) continue;
        if (tc::mbar_try_wait_ns(bar, parity, 1000)) break;
        if (*abort_flag) ok = false;
        else if (++polls > (1 << 21)) {                             // bounded: seconds
          if (lane == 0) atomicAdd(&tc::g_tc_timeouts, 1);
          *abort_flag = 1;
          ok = false;
        }
      }
    };
    while (refill()) {}

    // ---- MMAs ----
    struct Cursor { int item, u, nb; };
    // Moves a cursor to the stream's next item that has work (rows for this tile and encoder positions).
    auto seek = [&](Cursor& c) {
      c.u = 0; c.nb = 0;
      while (c.item < p.total_items) {
        const MsItem it = ms_item(p, c.item);
        if (tile < it.ntiles && it.nb > 0) { c.nb = it.nb; return; }
        c.item += item_step;
      }
    };
    Cursor cs = {2 * (int)blockIdx.x + hf, 0, 0}, cp = cs;
    uint32_t kc = 0, vc = 0;                      // blocks whose S / whose P V has been issued (ring slot = count % stages)
    uint32_t qs = 0;                              // Q tiles started by the S cursor (buffer = qs & 1)
    uint32_t pw = 0;                              // p_full phases consumed
    seek(cs);
    seek(cp);
    auto wait_s_operands = [&]() {
      if (cs.u == 0) wait_refilling(q_full + 2 * s + (qs & 1), (qs >> 1) & 1);
      wait_refilling(kvf + kc % kMsStages, (kc / kMsStages) & 1);
    };
    auto fire_s = [&]() {                         // elected lane
      const uint64_t qd = q_desc0 + (uint64_t)(((qs & 1) * kMsQBytes) >> 4);
      const uint64_t kd = k_desc0 + (uint64_t)(((kc % kMsStages) * 2 * kMsKVBytes) >> 4);
      tc::mma_ss_c<false>(tmem_s, qd, kd, idesc_s);
      tc::mma_ss_c<true>(tmem_s, qd + 2, kd + 2, idesc_s);
      tc::mma_ss_c<true>(tmem_s, qd + 4, kd + 4, idesc_s);
      tc::mma_ss_c<true>(tmem_s, qd + 6, kd + 6, idesc_s);
      tc::mma_commit(s_full + s);
    };
    auto advance_s = [&]() {
      ++kc;
      if (++cs.u == cs.nb) { ++qs; cs.item += item_step; seek(cs); }
    };
    if (cs.nb) {
      wait_s_operands();
      if (ok) {
        tc::tc_fence_after();
        if (tc::elect_one()) fire_s();
        __syncwarp();
        advance_s();
      }
    }
    while (ok && cp.nb) {
      // Operand waits first (normally long satisfied), so that nothing but the MMAs themselves stands
      // between the arrival of P(u) and the completion of S(u + 1).
      const int u = cp.u;
      const bool with_s = cs.nb != 0;
      if (with_s) wait_s_operands();
      wait_refilling(p_full + s, pw & 1);
      if (!ok) break;
      ++pw;
      tc::tc_fence_after();
      const uint32_t slot = vc % kMsStages;
      if (tc::elect_one()) {
        const uint64_t vd = v_desc0 + (uint64_t)((slot * 2 * kMsKVBytes) >> 4);
        if (u == 0) tc::mma_ts_c<false>(tmem_o, tmem_s, vd, idesc_o);
        else tc::mma_ts_c<true>(tmem_o, tmem_s, vd, idesc_o);
        tc::mma_ts_c<true>(tmem_o, tmem_s + 8, vd + 128, idesc_o);
        tc::mma_ts_c<true>(tmem_o, tmem_s + 16, vd + 256, idesc_o);
        tc::mma_ts_c<true>(tmem_o, tmem_s + 24, vd + 384, idesc_o);
        tc::mma_commit(kve + slot);                              // K (read by S(u)) and V of the block are done with
        if (u == cp.nb - 1) tc::mma_commit(o_full + s);
        if (with_s) fire_s();
      }
      __syncwarp();
      ++vc;
      if (++cp.u == cp.nb) { cp.item += item_step; seek(cp); }
      if (with_s) advance_s();
    }
    // loads still outstanding for the half's other stream (it may lag behind this one)
    {
      int polls = 0;
      while (ok && (lq_item < p.total_items || (tile == 0 && lk_item < p.total_items))) {
        if (refill()) { polls = 0; continue; }
        __nanosleep(500);
        if (*abort_flag || ++polls > (1 << 22)) ok = false;
      }
    }
  } else {
    // ---------------- softmax: four warps per stream ----------------
    const int q = warp & 3;                       // TMEM lane quarter = query rows 32 q .. 32 q + 31 of the tile
    const int s = warp >> 2;                      // stream
    const int hf = s >> 1, tile = s & 1;
    const int row = q * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    const uint32_t tmem_s = tmem_base + 64 * s + lane_addr;
    const uint32_t tmem_o = tmem_base + 256 + 64 * s + lane_addr;
    uint32_t g = 0;                               // blocks done
    uint32_t ow = 0;                              // o_full phases passed
    uint32_t qn = 0;                              // items with work so far (Q buffer = qn & 1)
    int release = -1;                             // Q buffer whose output stores are still to be waited for
    bool ok = true;
    // Once the output rows staged in a Q buffer have been read by the TMA store, the buffer goes back
    // to the producer (one arrival per softmax warp).
    auto release_q = [&]() {
      if (release >= 0) {
        if (lane == 0) { tc::bulk_wait_read<0>(); tc::mbar_arrive(q_empty + 2 * s + release); }
        release = -1;
      }
    };
    for (int item = 2 * (int)blockIdx.x + hf; ok && item < p.total_items; item += item_step) {
      const MsItem it = ms_item(p, item);
      if (tile >= it.ntiles) continue;
      const int m = it.row0 + tile * kMsBM + row;
      const bool row_live = m < p.M;
      const int64_t r_out = (int64_t)it.b * p.M + (row_live ? m : 0);
      if (it.nb == 0) {
        // no encoder position: the attention output is defined as zero
        if (row_live) {
          uint4* dst = reinterpret_cast<uint4*>(p.out + r_out * p.out_row_stride + it.h * kMsDH);
#pragma unroll
          for (int e = 0; e < 8; ++e) dst[e] = make_uint4(0u, 0u, 0u, 0u);
          if (p.lse != nullptr) p.lse[r_out * p.H + it.h] = -INFINITY;
        }
        continue;
      }
      float m_run = -INFINITY, l_run = 0.f;
      for (int u = 0; u < it.nb; ++u, ++g) {
        ok = tc::mbar_wait_likely_done(s_full + s, g & 1, abort_flag);
        if (!ok) break;
        tc::tc_fence_after();
        uint32_t r[kMsBN];
#pragma unroll
        for (int c = 0; c < kMsBN; c += 32) tc::tmem_ld32(tmem_s + c, *reinterpret_cast<uint32_t(*)[32]>(&r[c]));
        tc::tmem_ld_wait();
        const int valid = it.T - u * kMsBN;                         // positions of this block that exist (>= 1)
        if (valid < kMsBN) {
#pragma unroll
          for (int c = 0; c < kMsBN; ++c)
            if (c >= valid) r[c] = 0xff800000u;                     // -inf: no weight, no influence on the maximum
        }
        float mx0 = ms_max3(__uint_as_float(r[0]), __uint_as_float(r[1]), __uint_as_float(r[2]));
        float mx1 = ms_max3(__uint_as_float(r[3]), __uint_as_float(r[4]), __uint_as_float(r[5]));
        float mx2 = ms_max3(__uint_as_float(r[6]), __uint_as_float(r[7]), __uint_as_float(r[8]));
        float mx3 = ms_max3(__uint_as_float(r[9]), __uint_as_float(r[10]), __uint_as_float(r[11]));
#pragma unroll
        for (int c = 12; c + 7 < kMsBN; c += 8) {
          mx0 = ms_max3(mx0, __uint_as_float(r[c]), __uint_as_float(r[c + 1]));
          mx1 = ms_max3(mx1, __uint_as_float(r[c + 2]), __uint_as_float(r[c + 3]));
          mx2 = ms_max3(mx2, __uint_as_float(r[c + 4]), __uint_as_float(r[c + 5]));
          mx3 = ms_max3(mx3, __uint_as_float(r[c + 6]), __uint_as_float(r[c + 7]));
        }
        mx0 = ms_max3(mx0, __uint_as_float(r[kMsBN - 4]), __uint_as_float(r[kMsBN - 3]));
        mx1 = ms_max3(mx1, __uint_as_float(r[kMsBN - 2]), __uint_as_float(r[kMsBN - 1]));
        const float m_blk = fmaxf(ms_max3(mx0, mx1, mx2), mx3) * p.scale_log2;
        // The accumulator is rescaled only when the row maximum grows by more than 2^16 over the
        // reference in use (probabilities may then reach 65536, which bf16 and the fp32 sums hold
        // without loss of precision); with scores of ordinary spread that never happens after the
        // first sub-block.
        const bool grow = m_blk > m_run + kMsGrowLog2;              // always true on the first sub-block
        const float m_new = grow ? m_blk : m_run;
        const float alpha = grow ? ms_ex2(m_run - m_new) : 1.0f;    // 0 on the first sub-block
        m_run = m_new;
        if (u > 0 && __any_sync(kFullMask, grow)) {
          // O changes under the tensor core only here; P V of block u - 1 is complete, because this
          // block's S was issued after it and has been waited for.
#pragma unroll
          for (int c = 0; c < kMsDH; c += 16) {
            uint32_t o[16];
            tc::tmem_ld16(tmem_o + c, o);
            tc::tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tc::tmem_st16(tmem_o + c, o);
          }
        }
        const float neg_m = -m_new;
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
        for (int c = 0; c < kMsBN / 4; ++c) {
          const float e0 = ms_ex2(fmaf(__uint_as_float(r[4 * c]), p.scale_log2, neg_m));
          const float e1 = ms_ex2(fmaf(__uint_as_float(r[4 * c + 1]), p.scale_log2, neg_m));
          const float e2 = ms_ex2(fmaf(__uint_as_float(r[4 * c + 2]), p.scale_log2, neg_m));
          const float e3 = ms_ex2(fmaf(__uint_as_float(r[4 * c + 3]), p.scale_log2, neg_m));
          s0 += e0; s1 += e1; s2 += e2; s3 += e3;
          r[2 * c] = pack_bf16x2(e0, e1);
          r[2 * c + 1] = pack_bf16x2(e2, e3);
        }
        l_run = fmaf(l_run, alpha, (s0 + s1) + (s2 + s3));
#pragma unroll
        for (int c = 0; c < kMsBN / 2; c += 16) tc::tmem_st16(tmem_s + c, *reinterpret_cast<uint32_t(*)[16]>(&r[c]));
        tc::tmem_st_wait();
        tc::tc_fence_before();
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(p_full + s);
        if (u == 0) release_q();                  // the previous item's output stores have long been read
      }
      if (!ok) break;
      // ---- end of the item: O / l -> bf16 rows, staged in the item's Q tile, TMA store per warp ----
      ok = tc::mbar_wait(o_full + s, ow & 1, abort_flag);
      if (!ok) break;
      ++ow;
      tc::tc_fence_after();
      const uint32_t qb = qn & 1;
      ++qn;
      const float inv = 1.f / l_run;
      uint8_t* stage_row = q_tiles + (2 * s + qb) * kMsQBytes + row * 128;     // 128-byte swizzle: chunk j of row r at j ^ (r & 7)
#pragma unroll
      for (int c = 0; c < kMsDH; c += 32) {
        uint32_t o[32];
        tc::tmem_ld32(tmem_o + c, o);
        tc::tmem_ld_wait();
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const uint4 w = make_uint4(
              pack_bf16x2(__uint_as_float(o[8 * e]) * inv, __uint_as_float(o[8 * e + 1]) * inv),
              pack_bf16x2(__uint_as_float(o[8 * e + 2]) * inv, __uint_as_float(o[8 * e + 3]) * inv),
              pack_bf16x2(__uint_as_float(o[8 * e + 4]) * inv, __uint_as_float(o[8 * e + 5]) * inv),
              pack_bf16x2(__uint_as_float(o[8 * e + 6]) * inv, __uint_as_float(o[8 * e + 7]) * inv));
          *reinterpret_cast<uint4*>(stage_row + (((c / 8 + e) ^ (row & 7)) << 4)) = w;
        }
      }
      // The next item's first P V overwrites O; it is issued only after this stream's four warps have
      // arrived on p_full, i.e. after these loads.
      tc::tc_fence_before();
      tc::fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0 && it.row0 + tile * kMsBM + q * 32 < p.M) {
        tc::tma_store_4d(&map_o, q_tiles + (2 * s + qb) * kMsQBytes + q * 32 * 128, 0, it.h, it.row0 + tile * kMsBM + q * 32, it.b);
        tc::bulk_commit();
      }
      release = (int)qb;
      if (row_live && p.lse != nullptr) p.lse[r_out * p.H + it.h] = (m_run + log2f(l_run)) * 0.6931471805599453f;
    }
    if (lane == 0) tc::bulk_wait_all();           // shared memory stays valid until the last stores have read it
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == kMsSoftmaxWarps) tc::tmem_dealloc(tmem_base, 512);
}

inline bool cross_attn_ms_supported(int B, int M, int H, int d_h, int T_ctx) {
  return d_h == 64 && H <= 65535 && B <= 65535 && T_ctx >= 1 && M >= 1;
}

inline grace_status_t launch_cross_attn_ms(const uint16_t* q, int64_t q_row_stride, const uint16_t* k,
                                           const uint16_t* v, int64_t kv_stride_b, int64_t kv_stride_h,
                                           int64_t kv_stride_t, uint16_t* out, int64_t out_row_stride, float* lse,
                                           const int32_t* enc_len, int B, int M, int H, int T_ctx, float scale,
                                           cudaStream_t s) {
  CUtensorMap mq, mk, mv, mo;
  {
    const uint64_t dims[4] = {(uint64_t)kMsDH, (uint64_t)H, (uint64_t)M, (uint64_t)B};
    const uint64_t str[3] = {(uint64_t)kMsDH, (uint64_t)q_row_stride, (uint64_t)M * (uint64_t)q_row_stride};
    const uint32_t box[4] = {64u, 1u, (uint32_t)kMsBM, 1u};
    if (!tc::make_tmap_bf16(&mq, q, 4, dims, str, box)) return GRACE_CUDA_ERROR;
    const uint64_t ostr[3] = {(uint64_t)kMsDH, (uint64_t)out_row_stride, (uint64_t)M * (uint64_t)out_row_stride};
    const uint32_t obox[4] = {64u, 1u, 32u, 1u};                       // one softmax warp's rows
    if (!tc::make_tmap_bf16(&mo, out, 4, dims, ostr, obox)) return GRACE_CUDA_ERROR;
  }
  {
    const uint64_t dims[4] = {(uint64_t)kMsDH, (uint64_t)T_ctx, (uint64_t)H, (uint64_t)B};
    const uint64_t str[3] = {(uint64_t)kv_stride_t, (uint64_t)kv_stride_h, (uint64_t)kv_stride_b};
    const uint32_t box[4] = {64u, (uint32_t)kMsBN, 1u, 1u};
    if (!tc::make_tmap_bf16(&mk, k, 4, dims, str, box)) return GRACE_CUDA_ERROR;
    if (!tc::make_tmap_bf16(&mv, v, 4, dims, str, box)) return GRACE_CUDA_ERROR;
  }
  static unsigned long long attr_set_devices = 0;
  static int n_sm_of[kMaxDevices] = {0};
  DeviceSetup su(&attr_set_devices);
  if (su) {
    GRACE_CUDA_TRY(cudaFuncSetAttribute(cross_attn_ms_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMsSmemBytes));
    GRACE_CUDA_TRY(cudaDeviceGetAttribute(&n_sm_of[su.dev], cudaDevAttrMultiProcessorCount, su.dev));
    su.done();
  }
  const int n_sm = n_sm_of[su.dev];
  CrossMsParams p;
  p.out = out; p.lse = lse; p.enc_len = enc_len; p.out_row_stride = out_row_stride;
  p.B = B; p.M = M; p.H = H; p.T = T_ctx;
  p.pairs_m = (M + 2 * kMsBM - 1) / (2 * kMsBM);
  const int64_t items = (int64_t)p.pairs_m * H * B;
  if (items > 0x3fffffff) return GRACE_UNSUPPORTED_SHAPE;
  p.total_items = (int)items;
  p.scale_log2 = scale * 1.4426950408889634f;
  const int64_t ctas = (items + 1) / 2;
  const int grid = (int)(ctas < n_sm ? ctas : n_sm);
  launch_pdl(cross_attn_ms_kernel, dim3(grid), dim3(kMsThreads), kMsSmemBytes, s, mq, mk, mv, mo, p);
  GRACE_LAUNCH_CHECK();
  return GRACE_OK;
}

}  // namespace grace
