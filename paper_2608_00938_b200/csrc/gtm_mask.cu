// CD + GTM mask with score add (Sections 3.1, 4.1, 5.4) and the beam-state update after top-k
// (Sections 3.3, 4.4).
//
// One warp owns one beam row.  The row's child bitmask (V/64 words, one word per lane) and a warp
// prefix sum of its popcounts give every lane the k-th catalog-valid child directly, so matcher
// work (node-eligibility bit or Bloom probes) is done only for valid children and with all lanes
// busy.  The row is then streamed with float4 accesses: 512-byte warp stores out, and log-prob
// sectors in only where a token is allowed.  HBM-bound at the root levels (4 bytes out plus up to
// 4 bytes in per candidate); with the Bloom matcher the random 8-byte probes into the request's
// 512 KB filter (L2-resident) add a latency/L2-bandwidth term.
#include <cstdlib>
#include "common.cuh"

namespace grace {

struct MaskParams {
  const float* logp;
  const float* beam_score;
  const int32_t* beam_node;
  const uint64_t* beam_key;
  const uint64_t* child_bits;
  const int32_t* child_base;
  const uint64_t* matcher_bits;
  float* cand;
  float* row_lse;            // LOGITS mode: receives log-sum-exp of each live row
  const float2* lse_part;    // LOGITS mode, optional: [R][n_parts] (maximum, sum of e^(x - maximum)) per column tile,
  int n_parts;               //   left by the GEMM that produced the logits; the row is then not read for its sum
  uint64_t* allow_bits;
  int32_t* d_status;
  int64_t num_internal, num_nodes, words_per_request;
  int R, M, V, prefix_len;
  int bloom_mask_bits;     // 2^log2_bits - 1 (as uint32)
  int bloom_hashes;
};

// Position of the n-th (0-based) set bit of a 64-bit word that has more than n bits set.
__device__ __forceinline__ int nth_set_bit64(uint64_t word, int n) {
  uint32_t x = (uint32_t)word;
  int pos = 0;
  int c = __popc(x);
  if (n >= c) { n -= c; x = (uint32_t)(word >> 32); pos = 32; }
#pragma unroll
  for (int width = 16; width >= 1; width >>= 1) {
    const uint32_t low = x & ((1u << width) - 1u);
    c = __popc(low);
    if (n >= c) { n -= c; x >>= width; pos += width; } else { x = low; }
  }
  return pos;
}

constexpr int kMaskWarpsPerBlock = 8;
constexpr int kMaskSplitWarps = 32;      // SPLIT: warps that share one row (a CTA of 1024 threads)

// The log-sum-exp of a row from per-lane (maximum, sum of e^(x - maximum)) pairs (lanes without a pair pass
// (-inf, 0)): every lane returns the same value.  One definition, with the roundings spelled out, for the mask
// kernel and the merge kernel below, so that both give the same bits.
// G: lanes that share a row (32, or fewer when the pairs of several rows sit side by side in a warp).  Lanes
// without a pair contribute max(., -inf) and + 0, both exact, so the result does not depend on G.
template <int G = 32>
__device__ __forceinline__ float warp_merge_lse(float m_l, float s_l) {
  float m_w = m_l;
#pragma unroll
  for (int o = G / 2; o > 0; o >>= 1) m_w = fmaxf(m_w, __shfl_xor_sync(kFullMask, m_w, o));
  float s_w = (m_l > -INFINITY) ? __fmul_rn(s_l, expf(m_l - m_w)) : 0.f;
#pragma unroll
  for (int o = G / 2; o > 0; o >>= 1) s_w = __fadd_rn(s_w, __shfl_xor_sync(kFullMask, s_w, o));
  return __fadd_rn(m_w, logf(s_w));
}

// One warp per beam row, two phases per chunk of 2048 tokens:
//   1. the catalog-valid children (set bits of the node's child bitmask) are enumerated compactly,
//      lane k takes the k-th, (k+32)-th, ... child, evaluates the request's matcher for it and ORs
//      the result into the warp's allow words in shared memory.  Bloom probes are issued one at a
//      time and stop at the first clear bit (fewest L2 sectors; other rows' warps cover the latency).
//   2. the row is streamed: cand = score + logp where allowed, -inf elsewhere; a 32-byte sector of
//      log-probabilities is read only if one of its tokens is allowed.
// LOGITS = true: `logp` holds raw logits; the row's log-sum-exp is taken in a first streaming pass
// and cand = score + (logit - lse) for allowed tokens.
// SPLIT = true (few rows, e.g. step 0 with one beam per request): the 32 warps of a 1024-thread CTA share ONE
// row: each takes every 32nd group of 32 children in phase 1 and every 32nd group of 128 tokens in
// the streaming passes; the warp-level synchronisation points become CTA barriers.
template <int KIND, bool LOGITS, bool SPLIT>
__global__ void __launch_bounds__((SPLIT ? kMaskSplitWarps : kMaskWarpsPerBlock) * 32)
gtm_mask_kernel(const MaskParams p) {
  __shared__ uint64_t s_words[kMaskWarpsPerBlock][32];
  __shared__ unsigned long long s_allow[kMaskWarpsPerBlock][32];
  __shared__ int s_incl[kMaskWarpsPerBlock][32];
  __shared__ float s_lse[2][kMaskSplitWarps];
  pdl_wait();
  pdl_trigger();
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int r = SPLIT ? (int)blockIdx.x : (int)blockIdx.x * kMaskWarpsPerBlock + wib;
  if (r >= p.R) return;
  const int part = SPLIT ? wib : 0;                      // this warp's share of the row's work
  constexpr int kParts = SPLIT ? kMaskSplitWarps : 1;
  auto sync_row = [&]() { if (SPLIT) __syncthreads(); else __syncwarp(); };
  const int V = p.V;
  const int W = V >> 6;
  const int b = r / p.M;
  int node = __ldg(p.beam_node + r);
  bool dead = node < 0;
  if (!dead && node >= p.num_internal) {           // leaf or garbage: nothing below it
    if (node >= p.num_nodes && lane == 0) flag_status(p.d_status, GRACE_DEV_BAD_INDEX);
    dead = true;
  }
  const float score = p.beam_score != nullptr ? __ldg(p.beam_score + r) : 0.f;    // not needed for allow bits alone
  const uint64_t row_key = (KIND == GRACE_MATCH_PREFIX_BLOOM) ? __ldg(p.beam_key + r) : 0ull;
  const uint64_t* req_bits = (KIND == GRACE_MATCH_NONE) ? nullptr : p.matcher_bits + (int64_t)b * p.words_per_request;
  const int32_t base = dead ? -1 : __ldg(p.child_base + node);
  const float ninf = __int_as_float(0xff800000);
  const float* lrow = p.logp + (int64_t)r * V;
  bool saw_nan = false;
  float lse = 0.f;
  if (LOGITS && !dead) {
    // one streaming pass over the row: per-lane running maximum and rescaled sum, merged across the
    // warp at the end (the row is not kept: phase 2 re-reads only the allowed sectors, from L2)
    float m_l = -INFINITY, s_l = 0.f;
    const int n4 = V >> 2;
    if (p.lse_part != nullptr) {                           // the producer of the logits already summed each column tile
      if (part == 0 && lane < p.n_parts) {
        const float2 pr = __ldg(p.lse_part + (int64_t)r * p.n_parts + lane);
        m_l = pr.x;
        s_l = pr.y;
      }
    } else
    for (int c0 = part * 128; c0 < n4; c0 += kParts * 128) {
      float4 x[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int c = c0 + u * 32 + lane;
        x[u] = (c < n4) ? __ldg(reinterpret_cast<const float4*>(lrow) + c)
                        : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
      }
      float mx = m_l;
#pragma unroll
      for (int u = 0; u < 4; ++u) mx = fmaxf(mx, fmaxf(fmaxf(x[u].x, x[u].y), fmaxf(x[u].z, x[u].w)));
      if (mx > -INFINITY) {
        float acc = s_l * expf(m_l - mx);
#pragma unroll
        for (int u = 0; u < 4; ++u)
          acc += expf(x[u].x - mx) + expf(x[u].y - mx) + expf(x[u].z - mx) + expf(x[u].w - mx);
        s_l = acc;
        m_l = mx;
      }
    }
    if (!SPLIT) {
      lse = warp_merge_lse(m_l, s_l);
    } else {
      float m_w = m_l;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m_w = fmaxf(m_w, __shfl_xor_sync(kFullMask, m_w, o));
      float s_w = (m_l > -INFINITY) ? s_l * expf(m_l - m_w) : 0.f;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s_w += __shfl_xor_sync(kFullMask, s_w, o);
      if (lane == 0) { s_lse[0][wib] = m_w; s_lse[1][wib] = s_w; }
    }
  }
  if (SPLIT && LOGITS) {                                 // merge the warps' (maximum, rescaled sum) pairs
    __syncthreads();
    if (!dead) {
      float m_c = -INFINITY;
      for (int w = 0; w < kParts; ++w) m_c = fmaxf(m_c, s_lse[0][w]);
      float s_c = 0.f;
      for (int w = 0; w < kParts; ++w)
        if (s_lse[0][w] > -INFINITY) s_c += s_lse[1][w] * expf(s_lse[0][w] - m_c);
      lse = m_c + logf(s_c);
    }
  }
  if (LOGITS && lane == 0 && part == 0 && p.row_lse != nullptr) p.row_lse[r] = lse;
  uint64_t* words = s_words[SPLIT ? 0 : wib];
  unsigned long long* allow = s_allow[SPLIT ? 0 : wib];
  int* incl = s_incl[SPLIT ? 0 : wib];

  int rank_before_chunk = 0;
  for (int w0 = 0; w0 < W; w0 += 32) {
    uint64_t word = 0;
    if (!dead && w0 + lane < W) word = __ldg(p.child_bits + (int64_t)node * W + w0 + lane);
    const int pc = __popcll(word);
    int inc = pc;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int o = __shfl_up_sync(kFullMask, inc, d);
      if (lane >= d) inc += o;
    }
    const int total = __shfl_sync(kFullMask, inc, 31);
    sync_row();
    if (part == 0) {
      words[lane] = word;
      incl[lane] = inc;
      allow[lane] = (KIND == GRACE_MATCH_NONE) ? word : 0ull;
    }
    sync_row();

    if (KIND == GRACE_MATCH_NODE_BITMASK) {
      // The children of a node have consecutive ids, so the eligibility bits of this lane's
      // children are `pc` consecutive bits of the request's node bitmask; they are spread back
      // onto the set bits of the child word (a software bit-deposit), one lane per word.
      const int64_t first = (int64_t)base + rank_before_chunk + (inc - pc);
      uint64_t elig = 0ull;
      if (pc != 0 && first >= 0 && first + pc <= p.num_nodes) {
        const uint64_t lo = __ldg(req_bits + (first >> 6));
        const int sh = (int)(first & 63);
        elig = lo >> sh;
        if (sh != 0 && sh + pc > 64) elig |= __ldg(req_bits + (first >> 6) + 1) << (64 - sh);
      }
      uint64_t out = 0ull, rest = word;
      while (rest != 0ull) {
        const uint64_t low = rest & (0ull - rest);
        if (elig & 1ull) out |= low;
        elig >>= 1;
        rest ^= low;
      }
      if (part == 0) allow[lane] = out;
      sync_row();
    } else if (KIND != GRACE_MATCH_NONE) {
      for (int k0 = part * 32; k0 < total; k0 += kParts * 32) {
        const int k = k0 + lane;
        const bool have = k < total;
        // word holding the k-th child: smallest w with incl[w] > k
        int lo = 0;
#pragma unroll
        for (int step = 16; step >= 1; step >>= 1)
          if (have && incl[lo + step - 1] <= k) lo += step;
        const uint64_t cw = have ? words[lo] : 1ull;
        const int within = have ? k - (incl[lo] - __popcll(cw)) : 0;
        const int bit = nth_set_bit64(cw, within);
        bool ok = have;
        if (KIND == GRACE_MATCH_NODE_BITMASK) {
          const int64_t child = (int64_t)base + rank_before_chunk + k;
          if (ok) ok = (child >= 0 && child < p.num_nodes) && ((__ldg(req_bits + (child >> 6)) >> (child & 63)) & 1ull);
        } else {
          const int v = (w0 << 6) + (lo << 6) + bit;
          const uint64_t z = mix64(row_key | ((uint64_t)(v + 1) << (16 * p.prefix_len)));
          const uint32_t h1 = (uint32_t)z, h2 = (uint32_t)(z >> 32) | 1u;
          // One probe at a time, stopping at the first clear bit: the kernel is bound by the number of 32-byte
          // sectors it pulls out of L2 (probes are random within a 512 KB filter), not by their latency: probing
          // in pairs fetched 2.7 sectors per candidate instead of 2.25 and ran 10 % slower, all four at once 40 %.
          for (int i = 0; i < p.bloom_hashes && ok; ++i) {
            const uint32_t pos = (h1 + (uint32_t)i * h2) & (uint32_t)p.bloom_mask_bits;
            ok = (__ldg(req_bits + (pos >> 6)) >> (pos & 63)) & 1ull;
          }
        }
        if (ok) atomicOr(&allow[lo], 1ull << bit);
      }
      sync_row();
    }
    rank_before_chunk += total;

    if (p.allow_bits != nullptr && part == 0 && w0 + lane < W) p.allow_bits[(int64_t)r * W + w0 + lane] = allow[lane];
    if (p.cand != nullptr) {
      const int chunk_tokens = min(2048, V - (w0 << 6));
      // 128 tokens per iteration: lane handles tokens 4*lane .. 4*lane+3 of the group
      for (int g = part * 128; g < chunk_tokens; g += kParts * 128) {
        const int tok_in_chunk = g + 4 * lane;
        if (tok_in_chunk >= chunk_tokens) continue;           // V % 64 == 0, so all 4 or none
        const uint32_t nib = (uint32_t)(allow[tok_in_chunk >> 6] >> (tok_in_chunk & 63)) & 0xfu;
        // log-probs are read only where a token of this lane is allowed
        float4 lp = make_float4(0.f, 0.f, 0.f, 0.f);
        if (nib != 0u) {
          lp = __ldg(reinterpret_cast<const float4*>(lrow + (w0 << 6) + tok_in_chunk));
          if (LOGITS) lp = make_float4(lp.x - lse, lp.y - lse, lp.z - lse, lp.w - lse);
        }
        const float vals[4] = {lp.x, lp.y, lp.z, lp.w};
        float outv[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const bool okj = (nib >> j) & 1u;
          outv[j] = okj ? (score + vals[j]) : ninf;
          if (okj && vals[j] != vals[j]) saw_nan = true;
        }
        *reinterpret_cast<float4*>(p.cand + (int64_t)r * V + (w0 << 6) + tok_in_chunk) =
            make_float4(outv[0], outv[1], outv[2], outv[3]);
      }
    }
    sync_row();
  }
  if (saw_nan) flag_status(p.d_status, GRACE_DEV_NAN);
}

// ---------------------------------------------------------------------------------------------
// The allow bits of the prefix-Bloom matcher with the request's filter in distributed shared memory.
// The probes of the kernel above are random 8-byte reads in a 512 KB filter that lives in L2: the kernel is
// bound by the 32-byte sectors it pulls from there.  Here a cluster of kBloomClusterCtas CTAs serves ONE
// request: each CTA copies its share of the filter words into its shared memory once, and every probe is an
// ld.shared::cluster from the CTA that owns the word.  Same hash, same positions, same bits.
// grid (kBloomClusterCtas, B); the cluster's warps take the request's rows round-robin.
// MEASURED SLOWER than the L2 form and therefore off unless GRACE_BLOOM_DSMEM is set in the environment: at 32
// requests x 2048 rows x 2048 tokens (430 catalog children per row, filter 2^22 x 4) 796 us against 278 us;
// with four probes in flight per lane instead of one at a time 1184 us.  Time follows the number of probes
// (63 M and 113 M): random 8-byte loads from other SMs' shared memory run at about a third of a probe per
// clock and SM, the L2 serves 2.4 times that.  Kept as the record of that measurement.
// ---------------------------------------------------------------------------------------------
constexpr int kBloomClusterCtas = 4;
constexpr int kBloomClusterWarps = 16;                    // per CTA

__device__ __forceinline__ uint32_t mask_cluster_rank() {
  uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r;
}
__device__ __forceinline__ void mask_cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint64_t ld_cluster_u64(uint32_t local_smem_addr, uint32_t rank) {
  uint64_t v;
  asm volatile(
      "{\n\t.reg .b32 ra;\n\t"
      "mapa.shared::cluster.u32 ra, %1, %2;\n\t"
      "ld.shared::cluster.u64 %0, [ra];\n\t}"
      : "=l"(v) : "r"(local_smem_addr), "r"(rank) : "memory");
  return v;
}

__global__ void __launch_bounds__(kBloomClusterWarps * 32, 1)
gtm_allow_bloom_cluster_kernel(const MaskParams p, int log2_words_per_cta) {
  extern __shared__ __align__(16) uint64_t s_filter[];                         // this CTA's words of the request's filter
  __shared__ uint64_t s_words[kBloomClusterWarps][32];
  __shared__ unsigned long long s_allow[kBloomClusterWarps][32];
  __shared__ int s_incl[kBloomClusterWarps][32];
  pdl_wait();
  pdl_trigger();
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const uint32_t rank = mask_cluster_rank();
  const int b = blockIdx.y;
  const int words_per_cta = 1 << log2_words_per_cta;
  {
    const uint4* src = reinterpret_cast<const uint4*>(p.matcher_bits + (int64_t)b * p.words_per_request +
                                                     (int64_t)rank * words_per_cta);
    uint4* dst = reinterpret_cast<uint4*>(s_filter);
    for (int i = threadIdx.x; i < words_per_cta / 2; i += blockDim.x) dst[i] = __ldg(src + i);
  }
  __syncthreads();
  mask_cluster_sync();                                     // every share is in place before anyone probes
  const uint32_t filter_base = (uint32_t)__cvta_generic_to_shared(s_filter);
  const int V = p.V, W = V >> 6;
  uint64_t* words = s_words[wib];
  unsigned long long* allow = s_allow[wib];
  int* incl = s_incl[wib];
  for (int m = (int)rank * kBloomClusterWarps + wib; m < p.M; m += kBloomClusterCtas * kBloomClusterWarps) {
    const int r = b * p.M + m;
    int node = __ldg(p.beam_node + r);
    bool dead = node < 0;
    if (!dead && node >= p.num_internal) {
      if (node >= p.num_nodes && lane == 0) flag_status(p.d_status, GRACE_DEV_BAD_INDEX);
      dead = true;
    }
    const uint64_t row_key = __ldg(p.beam_key + r);
    for (int w0 = 0; w0 < W; w0 += 32) {
      uint64_t word = 0;
      if (!dead && w0 + lane < W) word = __ldg(p.child_bits + (int64_t)node * W + w0 + lane);
      const int pc = __popcll(word);
      int inc = pc;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(kFullMask, inc, d);
        if (lane >= d) inc += o;
      }
      const int total = __shfl_sync(kFullMask, inc, 31);
      __syncwarp();
      words[lane] = word;
      incl[lane] = inc;
      allow[lane] = 0ull;
      __syncwarp();
      for (int k0 = 0; k0 < total; k0 += 32) {
        const int k = k0 + lane;
        const bool have = k < total;
        int lo = 0;
#pragma unroll
        for (int step = 16; step >= 1; step >>= 1)
          if (have && incl[lo + step - 1] <= k) lo += step;
        const uint64_t cw = have ? words[lo] : 1ull;
        const int within = have ? k - (incl[lo] - __popcll(cw)) : 0;
        const int bit = nth_set_bit64(cw, within);
        const int v = (w0 << 6) + (lo << 6) + bit;
        const uint64_t z = mix64(row_key | ((uint64_t)(v + 1) << (16 * p.prefix_len)));
        const uint32_t h1 = (uint32_t)z, h2 = (uint32_t)(z >> 32) | 1u;
        bool ok = have;
        for (int i = 0; i < p.bloom_hashes && ok; ++i) {
          const uint32_t pos = (h1 + (uint32_t)i * h2) & (uint32_t)p.bloom_mask_bits;
          const uint32_t w = pos >> 6;
          const uint64_t fw = ld_cluster_u64(filter_base + ((w & (uint32_t)(words_per_cta - 1)) << 3), w >> log2_words_per_cta);
          ok = (fw >> (pos & 63)) & 1ull;
        }
        if (ok) atomicOr(&allow[lo], 1ull << bit);
      }
      __syncwarp();
      if (w0 + lane < W) p.allow_bits[(int64_t)r * W + w0 + lane] = allow[lane];
      __syncwarp();
    }
  }
  mask_cluster_sync();                                     // no CTA leaves while its share may still be probed
}

// The rows' log-sum-exp from the partials a logits GEMM left per 256-column tile, when the mask ran BEFORE that
// GEMM (allow bits first, so that the GEMM stores only allowed logits): one warp per row, the arithmetic of the
// mask kernel's own merge; dead rows (no node, or a leaf) get 0 as there.  G lanes per row, 32 / G rows per warp.
template <int G>
__global__ void __launch_bounds__(256)
row_lse_from_parts_kernel(const float2* __restrict__ lse_part, int n_parts, const int32_t* __restrict__ beam_node,
                          int64_t num_internal, float* __restrict__ row_lse, int R) {
  pdl_wait();
  pdl_trigger();
  const int lane = threadIdx.x & 31;
  const int part = lane % G;
  const int r = (blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * (32 / G) + lane / G;
  const bool in_range = r < R;                             // (whole warps stay: the merge shuffles over all lanes)
  const int node = in_range ? __ldg(beam_node + r) : -1;
  const bool dead = node < 0 || node >= num_internal;
  float m_l = -INFINITY, s_l = 0.f;
  if (!dead && part < n_parts) {
    const float2 pr = __ldg(lse_part + (int64_t)r * n_parts + part);
    m_l = pr.x;
    s_l = pr.y;
  }
  const float merged = warp_merge_lse<G>(m_l, s_l);
  if (in_range && part == 0) row_lse[r] = dead ? 0.f : merged;
}

// ---------------------------------------------------------------------------------------------
// CD + GTM lookup on the paper's index form (Sections 4.4, 5.4, Appendix A): CSR child entries
// with ids of deduplicated per-node bitmask / Bloom rows, tested against the request's rows.
// grid (ceil(M / 8), B): a CTA serves eight beams of ONE request, so the request's attribute
// bitmask and its N_loc location rows are staged in shared memory once and reused by every
// candidate of those beams.  One warp per beam; lanes take the child entries of the beam's node.
// Evaluation order as in the paper: bitmask first (stop at the first failing word), Bloom only for
// entries that pass, inner scan stops at the first word that is not contained, outer scan at the
// first location that is.
// ---------------------------------------------------------------------------------------------
struct LookupParams {
  const float* logp;
  const float* beam_score;
  const int32_t* beam_node;
  grace_gtm_index_t idx;
  float* cand;
  uint64_t* allow_bits;
  int32_t* d_status;
  int M;
};

constexpr int kLookupMaxWords = 64;          // V <= 4096

template <int WBM, int WBL>
__global__ void __launch_bounds__(kMaskWarpsPerBlock * 32)
gtm_lookup_kernel(const LookupParams p) {
  extern __shared__ uint64_t s_user[];                         // [WBM] bitmask, then [N_loc][WBL]
  __shared__ unsigned long long s_allow[kMaskWarpsPerBlock][kLookupMaxWords];
  __shared__ int s_queue[kMaskWarpsPerBlock][64];
  const grace_gtm_index_t& ix = p.idx;
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int b = blockIdx.y;
  const int V = ix.V, W = V >> 6;
  for (int i = threadIdx.x; i < WBM; i += blockDim.x) s_user[i] = ix.user_bitmask[(int64_t)b * WBM + i];
  for (int i = threadIdx.x; i < ix.N_loc * WBL; i += blockDim.x)
    s_user[WBM + i] = ix.user_blooms[(int64_t)b * ix.N_loc * WBL + i];
  __syncthreads();
  const int m = blockIdx.x * kMaskWarpsPerBlock + wib;
  if (m >= p.M) return;
  const int64_t r = (int64_t)b * p.M + m;
  unsigned long long* allow = s_allow[wib];
  for (int w = lane; w < W; w += 32) allow[w] = 0ull;
  __syncwarp();
  const int node = __ldg(p.beam_node + r);
  bool dead = node < 0;
  if (!dead && node >= ix.num_nodes) {
    if (lane == 0) flag_status(p.d_status, GRACE_DEV_BAD_INDEX);
    dead = true;
  }
  if (!dead) {
    const int e_start = __ldg(ix.node_offsets + node), e_end = __ldg(ix.node_offsets + node + 1);
    // With k-way partitioned rows the scan runs over the partition slots of the node's entries (one
    // contiguous range, since slots follow entry order); a slot that passes both tests keeps its entry.
    const bool kway = (ix.part_offsets != nullptr);
    const int start = kway ? __ldg(ix.part_offsets + e_start) : e_start;
    const int end = kway ? __ldg(ix.part_offsets + e_end) : e_end;
    int* queue = s_queue[wib];                 // slots that passed the bitmask, waiting for Bloom
    int queued = 0;
    for (int j0 = start; j0 < end || queued > 0; j0 += 32) {
      // ---- bitmask stage: one entry per lane, first failing word ends it ----
      const int j = j0 + lane;
      bool pass = false;
      if (j < end) {
        const uint64_t* bm = ix.bitmask_table + (int64_t)__ldg(ix.bitmask_index + j) * WBM;
        pass = true;
#pragma unroll
        for (int w = 0; w < WBM; ++w) {
          if (!pass) break;
          const uint64_t u = s_user[w];
          pass = (__ldg(bm + w) & u) == u;
        }
      }
      // survivors are queued so that the (much longer) Bloom stage always runs with full warps
      const uint32_t votes = __ballot_sync(kFullMask, pass);
      if (pass) queue[queued + __popc(votes & ((1u << lane) - 1u))] = j;
      queued += __popc(votes);
      __syncwarp();
      const bool last_round = (j0 + 32 >= end);
      while (queued >= 32 || (last_round && queued > 0)) {
        const int take = min(queued, 32);
        const int e = (lane < take) ? queue[queued - take + lane] : -1;
        queued -= take;
        bool ok = false;
        if (e >= 0) {
          const uint64_t* blp = ix.bloom_table + (int64_t)__ldg(ix.bloom_index + e) * WBL;
          uint64_t nbl[WBL];                   // complement of the candidate row: q is contained iff q & ~row == 0
#pragma unroll
          for (int w = 0; w < WBL; ++w) nbl[w] = ~__ldg(blp + w);
          // ANY-of-N_loc, branch-free inside a group of eight locations, early exit between groups
          for (int q0 = 0; q0 < ix.N_loc && !ok; q0 += 8) {
            const int qn = min(8, ix.N_loc - q0);
            for (int q = 0; q < qn; ++q) {
              const uint64_t* qr = s_user + WBM + (q0 + q) * WBL;
              uint64_t outside = 0ull;
#pragma unroll
              for (int w = 0; w < WBL; ++w) outside |= qr[w] & nbl[w];
              ok = ok || (outside == 0ull);
            }
          }
        }
        if (ok) {
          int entry = e;
          if (kway) {                          // the entry that owns slot e: last one whose first slot is <= e
            int lo = e_start, hi = e_end - 1;
            while (lo < hi) {
              const int mid = (lo + hi + 1) >> 1;
              if (__ldg(ix.part_offsets + mid) <= e) lo = mid; else hi = mid - 1;
            }
            entry = lo;
          }
          const int tok = (int)__ldg(ix.csr_tokens + entry);
          if (tok >= 0 && tok < V) atomicOr(&allow[tok >> 6], 1ull << (tok & 63));
        }
        __syncwarp();
      }
      if (j0 >= end) break;                    // only the final drain was left
    }
  }
  __syncwarp();
  const float score = __ldg(p.beam_score + r);
  const float ninf = __int_as_float(0xff800000);
  const float* lrow = p.logp + r * V;
  bool saw_nan = false;
  if (p.allow_bits != nullptr)
    for (int w = lane; w < W; w += 32) p.allow_bits[r * W + w] = allow[w];
  if (p.cand != nullptr) {
    for (int g = 0; g < V; g += 128) {
      const int tok0 = g + 4 * lane;
      if (tok0 >= V) continue;
      const uint32_t nib = (uint32_t)(allow[tok0 >> 6] >> (tok0 & 63)) & 0xfu;
      float4 lp = make_float4(0.f, 0.f, 0.f, 0.f);
      if (nib != 0u) lp = __ldg(reinterpret_cast<const float4*>(lrow + tok0));
      const float vals[4] = {lp.x, lp.y, lp.z, lp.w};
      float outv[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const bool okj = (nib >> j) & 1u;
        outv[j] = okj ? (score + vals[j]) : ninf;
        if (okj && vals[j] != vals[j]) saw_nan = true;
      }
      *reinterpret_cast<float4*>(p.cand + r * V + tok0) = make_float4(outv[0], outv[1], outv[2], outv[3]);
    }
  }
  if (saw_nan) flag_status(p.d_status, GRACE_DEV_NAN);
}

__global__ void beam_update_csr_kernel(const int32_t* __restrict__ parent, const int32_t* __restrict__ token,
                                       const float* __restrict__ score, const int32_t* __restrict__ prev_node,
                                       const uint64_t* __restrict__ prev_key, const grace_gtm_index_t ix,
                                       int32_t* __restrict__ new_node, uint64_t* __restrict__ new_key, int B, int K,
                                       int M_prev, int prefix_len, int32_t* d_status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B * K) return;
  const int b = i / K;
  const int par = parent[i], tok = token[i];
  if (par < 0 || par >= M_prev || tok < 0 || tok >= ix.V) {
    flag_status(d_status, GRACE_DEV_BAD_INDEX);
    new_node[i] = -1;
    new_key[i] = 0;
    return;
  }
  const int64_t src = (int64_t)b * M_prev + par;
  new_key[i] = prev_key[src] | ((uint64_t)(tok + 1) << (16 * prefix_len));
  const int node = prev_node[src];
  int out = -1;
  if (node >= 0 && node < ix.num_nodes && score[i] != __int_as_float(0xff800000)) {
    int lo = ix.node_offsets[node], hi = ix.node_offsets[node + 1];       // tokens are sorted inside the range
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      const int t = (int)ix.csr_tokens[mid];
      if (t < tok) lo = mid + 1; else hi = mid;
    }
    if (lo < ix.node_offsets[node + 1] && (int)ix.csr_tokens[lo] == tok) out = ix.csr_child_nodes[lo];
  }
  new_node[i] = out;
}

__global__ void beam_update_kernel(const int32_t* __restrict__ parent, const int32_t* __restrict__ token,
                                   const float* __restrict__ score, const int32_t* __restrict__ prev_node,
                                   const uint64_t* __restrict__ prev_key, const uint64_t* __restrict__ child_bits,
                                   const int32_t* __restrict__ child_base, int64_t num_internal,
                                   int32_t* __restrict__ new_node, uint64_t* __restrict__ new_key,
                                   int B, int K, int M_prev, int V, int prefix_len, int32_t* d_status) {
  pdl_wait();
  pdl_trigger();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B * K) return;
  const int b = i / K;
  int par = parent[i];
  const int tok = token[i];
  if (par < 0 || par >= M_prev || tok < 0 || tok >= V) {
    flag_status(d_status, GRACE_DEV_BAD_INDEX);
    new_node[i] = -1;
    new_key[i] = 0;
    return;
  }
  const int64_t src = (int64_t)b * M_prev + par;
  new_key[i] = prev_key[src] | ((uint64_t)(tok + 1) << (16 * prefix_len));
  const int node = prev_node[src];
  int out = -1;
  if (node >= 0 && node < num_internal && score[i] != __int_as_float(0xff800000)) {
    const int W = V >> 6;
    const uint64_t* row = child_bits + (int64_t)node * W;
    const uint64_t word = row[tok >> 6];
    if ((word >> (tok & 63)) & 1ull) {
      int rank = __popcll(word & ((1ull << (tok & 63)) - 1ull));
      for (int w = 0; w < (tok >> 6); ++w) rank += __popcll(row[w]);
      out = child_base[node] + rank;
    }
  }
  new_node[i] = out;
}

}  // namespace grace

static bool trie_ok(const grace_trie_t* t, int V) {
  return t && t->child_bits && t->child_base && t->V == V && V > 0 && V % 64 == 0 && V < 65535 &&
         t->num_internal > 0 && t->num_nodes >= t->num_internal && t->L >= 1 && t->L <= 4;
}

static grace_status_t launch_mask(const float* logp, bool logits, float* row_lse, const float* beam_score,
                                  const int32_t* beam_node, const uint64_t* beam_key, const grace_trie_t* trie,
                                  const grace_matcher_t* matcher, float* cand, uint64_t* allow_bits, int B, int M,
                                  int V, int prefix_len, int32_t* d_status, void* stream,
                                  const float* lse_part = nullptr, int n_parts = 0) {
  using namespace grace;
  const bool bits_only = (logp == nullptr);              // CD + matcher alone: no values in, allow bits out
  if (bits_only && (logits || cand || !allow_bits)) return GRACE_INVALID_ARG;
  if ((!bits_only && !beam_score) || !beam_node || !matcher || (!cand && !allow_bits)) return GRACE_INVALID_ARG;
  if (B <= 0 || M <= 0 || (int64_t)B * M > 0x7fffffff) return GRACE_INVALID_ARG;
  if (!trie_ok(trie, V)) return GRACE_INVALID_ARG;
  if (prefix_len < 0 || prefix_len >= trie->L) return GRACE_INVALID_ARG;
  if (!grace_aligned16(logp) || (cand && !grace_aligned16(cand))) return GRACE_INVALID_ARG;
  MaskParams p;
  p.logp = logp; p.beam_score = beam_score; p.beam_node = beam_node; p.beam_key = beam_key;
  p.child_bits = trie->child_bits; p.child_base = trie->child_base;
  p.matcher_bits = matcher->bits; p.cand = cand; p.row_lse = row_lse; p.allow_bits = allow_bits; p.d_status = d_status;
  if (lse_part != nullptr && (!logits || n_parts < 1 || n_parts > 32 || (reinterpret_cast<uintptr_t>(lse_part) & 7)))
    return GRACE_INVALID_ARG;
  p.lse_part = reinterpret_cast<const float2*>(lse_part); p.n_parts = n_parts;
  p.num_internal = trie->num_internal; p.num_nodes = trie->num_nodes;
  p.words_per_request = matcher->words_per_request;
  p.R = B * M; p.M = M; p.V = V; p.prefix_len = prefix_len;
  p.bloom_mask_bits = 0; p.bloom_hashes = 0;
  cudaStream_t s = (cudaStream_t)stream;
  // Plain launches (no early scheduling under the previous kernel's tail): starting this kernel's CTAs while the
  // logits GEMM drains made the dense trie level 0.3 ms slower in the decode loop.
  // few rows: a CTA per row, so that the row's matcher look-ups and its streaming passes use eight warps
  const bool split = p.R <= 2048;
  const int blocks = split ? p.R : (p.R + kMaskWarpsPerBlock - 1) / kMaskWarpsPerBlock;
  const int threads = (split ? kMaskSplitWarps : kMaskWarpsPerBlock) * 32;
#define GRACE_MASK_LAUNCH(K)                                                      \
  do {                                                                            \
    if (logits && split) gtm_mask_kernel<K, true, true><<<blocks, threads, 0, s>>>(p);        \
    else if (logits) gtm_mask_kernel<K, true, false><<<blocks, threads, 0, s>>>(p);           \
    else if (split) gtm_mask_kernel<K, false, true><<<blocks, threads, 0, s>>>(p);            \
    else gtm_mask_kernel<K, false, false><<<blocks, threads, 0, s>>>(p);                      \
  } while (0)
  switch (matcher->kind) {
    case GRACE_MATCH_NONE:
      GRACE_MASK_LAUNCH(GRACE_MATCH_NONE);
      break;
    case GRACE_MATCH_NODE_BITMASK:
      if (!matcher->bits || matcher->words_per_request * 64 < trie->num_nodes) return GRACE_INVALID_ARG;
      GRACE_MASK_LAUNCH(GRACE_MATCH_NODE_BITMASK);
      break;
    case GRACE_MATCH_PREFIX_BLOOM:
      if (!matcher->bits || !beam_key || matcher->bloom_log2_bits < 6 || matcher->bloom_log2_bits > 32 ||
          matcher->bloom_hashes < 1 || matcher->bloom_hashes > 16 ||
          matcher->words_per_request != (int64_t)((1ull << matcher->bloom_log2_bits) / 64))
        return GRACE_INVALID_ARG;
      p.bloom_mask_bits = (int)(uint32_t)((1ull << matcher->bloom_log2_bits) - 1ull);
      p.bloom_hashes = matcher->bloom_hashes;
      static const bool dsmem_filter = getenv("GRACE_BLOOM_DSMEM") != nullptr;    // measured slower: see the kernel
      if (dsmem_filter && bits_only && matcher->bloom_log2_bits >= 10 && matcher->bloom_log2_bits <= 22 && M >= 256 &&
          grace_aligned16(matcher->bits)) {
        // the request's filter in the shared memory of a cluster of four CTAs (up to 128 KB each)
        const int log2_words_per_cta = matcher->bloom_log2_bits - 6 - 2;
        const size_t smem = (size_t)8 << log2_words_per_cta;
        static unsigned long long attr_set_devices = 0;
        DeviceSetup su(&attr_set_devices);
        if (su) {
          GRACE_CUDA_TRY(cudaFuncSetAttribute(gtm_allow_bloom_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              128 * 1024));
          su.done();
        }
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = kBloomClusterCtas; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.gridDim = dim3(kBloomClusterCtas, B); cfg.blockDim = dim3(kBloomClusterWarps * 32);
        cfg.dynamicSmemBytes = smem; cfg.stream = s; cfg.attrs = attr; cfg.numAttrs = 2;
        GRACE_CUDA_TRY(cudaLaunchKernelEx(&cfg, gtm_allow_bloom_cluster_kernel, p, log2_words_per_cta));
        break;
      }
      GRACE_MASK_LAUNCH(GRACE_MATCH_PREFIX_BLOOM);
      break;
    default:
      return GRACE_INVALID_ARG;
  }
#undef GRACE_MASK_LAUNCH
  GRACE_LAUNCH_CHECK();
  return GRACE_OK;
}

extern "C" grace_status_t grace_gtm_mask(const float* logp, const float* beam_score,
                                         const int32_t* beam_node, const uint64_t* beam_key,
                                         const grace_trie_t* trie, const grace_matcher_t* matcher,
                                         float* cand, uint64_t* allow_bits, int B, int M, int V,
                                         int prefix_len, int32_t* d_status, void* stream) {
  return launch_mask(logp, false, nullptr, beam_score, beam_node, beam_key, trie, matcher, cand, allow_bits, B, M, V,
                     prefix_len, d_status, stream);
}

extern "C" grace_status_t grace_gtm_mask_logits(const float* logits, float* row_lse, const float* beam_score,
                                                const int32_t* beam_node, const uint64_t* beam_key,
                                                const grace_trie_t* trie, const grace_matcher_t* matcher,
                                                float* cand, uint64_t* allow_bits, int B, int M, int V,
                                                int prefix_len, int32_t* d_status, void* stream) {
  return launch_mask(logits, true, row_lse, beam_score, beam_node, beam_key, trie, matcher, cand, allow_bits, B, M, V,
                     prefix_len, d_status, stream);
}

extern "C" grace_status_t grace_gtm_mask_logits_parts(const float* logits, float* row_lse, const float* beam_score,
                                                const int32_t* beam_node, const uint64_t* beam_key,
                                                const grace_trie_t* trie, const grace_matcher_t* matcher,
                                                float* cand, uint64_t* allow_bits, int B, int M, int V,
                                                int prefix_len, const float* lse_part, int n_parts, int32_t* d_status,
                                                      void* stream) {
  return launch_mask(logits, true, row_lse, beam_score, beam_node, beam_key, trie, matcher, cand, allow_bits, B, M, V,
                     prefix_len, d_status, stream, lse_part, n_parts);
}

extern "C" grace_status_t grace_gtm_allow_bits(const int32_t* beam_node, const uint64_t* beam_key,
                                               const grace_trie_t* trie, const grace_matcher_t* matcher,
                                               uint64_t* allow_bits, int B, int M, int V, int prefix_len,
                                               int32_t* d_status, void* stream) {
  return launch_mask(nullptr, false, nullptr, nullptr, beam_node, beam_key, trie, matcher, nullptr, allow_bits, B, M, V,
                     prefix_len, d_status, stream);
}

extern "C" grace_status_t grace_row_lse_from_parts(const float* lse_part, int n_parts, const int32_t* beam_node,
                                                   const grace_trie_t* trie, float* row_lse, int R, void* stream) {
  if (!lse_part || !beam_node || !trie || !row_lse || R <= 0 || n_parts < 1 || n_parts > 32 ||
      (reinterpret_cast<uintptr_t>(lse_part) & 7))
    return GRACE_INVALID_ARG;
  const float2* parts = reinterpret_cast<const float2*>(lse_part);
  cudaStream_t s = (cudaStream_t)stream;
  const int64_t ni = trie->num_internal;
  if (n_parts <= 8)
    grace::launch_pdl(grace::row_lse_from_parts_kernel<8>, dim3((R + 31) / 32), dim3(256), 0, s, parts, n_parts, beam_node, ni, row_lse, R);
  else if (n_parts <= 16)
    grace::launch_pdl(grace::row_lse_from_parts_kernel<16>, dim3((R + 15) / 16), dim3(256), 0, s, parts, n_parts, beam_node, ni, row_lse, R);
  else
    grace::launch_pdl(grace::row_lse_from_parts_kernel<32>, dim3((R + 7) / 8), dim3(256), 0, s, parts, n_parts, beam_node, ni, row_lse, R);
  GRACE_LAUNCH_CHECK();
  return GRACE_OK;
}

extern "C" grace_status_t grace_beam_update(const int32_t* parent, const int32_t* token, const float* score,
                                            const int32_t* prev_node, const uint64_t* prev_key,
                                            const grace_trie_t* trie, int32_t* new_node, uint64_t* new_key,
                                            int B, int K, int M_prev, int prefix_len,
                                            int32_t* d_status, void* stream) {
  if (!parent || !token || !score || !prev_node || !prev_key || !new_node || !new_key) return GRACE_INVALID_ARG;
  if (!trie || !trie_ok(trie, trie->V)) return GRACE_INVALID_ARG;
  if (B <= 0 || K <= 0 || M_prev <= 0 || prefix_len < 0 || prefix_len >= 4) return GRACE_INVALID_ARG;
  const int n = B * K;
  grace::launch_pdl(grace::beam_update_kernel, dim3((n + 255) / 256), dim3(256), 0, (cudaStream_t)stream,
      parent, token, score, prev_node, prev_key, trie->child_bits, trie->child_base, trie->num_internal,
      new_node, new_key, B, K, M_prev, trie->V, prefix_len, d_status);
  GRACE_LAUNCH_CHECK();
  return GRACE_OK;
}

static bool gtm_index_ok(const grace_gtm_index_t* ix) {
  return ix && ix->node_offsets && ix->csr_child_nodes && ix->csr_tokens && ix->bitmask_index && ix->bloom_index &&
         ix->bitmask_table && ix->bloom_table && ix->V > 0 && ix->V % 64 == 0 && ix->V <= 32767 && ix->L >= 1 &&
         ix->L <= 4 && ix->num_nodes > 0 && ix->num_entries == ix->num_nodes - 1 && ix->W_bm >= 1 && ix->W_bl >= 1 &&
         ix->N_loc >= 0;
}

extern "C" grace_status_t grace_gtm_lookup(const float* logp, const float* beam_score, const int32_t* beam_node,
                                           const grace_gtm_index_t* index, float* cand, uint64_t* allow_bits,
                                           int B, int M, int32_t* d_status, void* stream) {
  using namespace grace;
  if (!logp || !beam_score || !beam_node || (!cand && !allow_bits) || !gtm_index_ok(index)) return GRACE_INVALID_ARG;
  if (!index->user_bitmask || (index->N_loc > 0 && !index->user_blooms)) return GRACE_INVALID_ARG;
  if (B <= 0 || M <= 0 || B > 65535) return GRACE_INVALID_ARG;
  if (index->V > 64 * kLookupMaxWords || index->N_loc > 256) return GRACE_UNSUPPORTED_SHAPE;
  if (!grace_aligned16(logp) || (cand && !grace_aligned16(cand))) return GRACE_INVALID_ARG;
  LookupParams p;
  p.logp = logp; p.beam_score = beam_score; p.beam_node = beam_node; p.idx = *index; p.cand = cand;
  p.allow_bits = allow_bits; p.d_status = d_status; p.M = M;
  dim3 grid((unsigned)((M + kMaskWarpsPerBlock - 1) / kMaskWarpsPerBlock), (unsigned)B);
  const size_t smem = (size_t)(index->W_bm + (size_t)index->N_loc * index->W_bl) * sizeof(uint64_t);
  cudaStream_t s = (cudaStream_t)stream;
  const int threads = kMaskWarpsPerBlock * 32;
  if (index->W_bm == 7 && index->W_bl == 4) gtm_lookup_kernel<7, 4><<<grid, threads, smem, s>>>(p);
  else if (index->W_bm == 2 && index->W_bl == 4) gtm_lookup_kernel<2, 4><<<grid, threads, smem, s>>>(p);
  else if (index->W_bm == 1 && index->W_bl == 1) gtm_lookup_kernel<1, 1><<<grid, threads, smem, s>>>(p);
  else if (index->W_bm == 4 && index->W_bl == 4) gtm_lookup_kernel<4, 4><<<grid, threads, smem, s>>>(p);
  else return GRACE_UNSUPPORTED_SHAPE;      // row widths are compile-time: (7,4) as in the paper, plus (1,1), (2,4), (4,4)
  GRACE_LAUNCH_CHECK();
  return GRACE_OK;
}

extern "C" grace_status_t grace_beam_update_csr(const int32_t* parent, const int32_t* token, const float* score,
                                                const int32_t* prev_node, const uint64_t* prev_key,
                                                const grace_gtm_index_t* index, int32_t* new_node, uint64_t* new_key,
                                                int B, int K, int M_prev, int prefix_len, int32_t* d_status,
                                                void* stream) {
  if (!parent || !token || !score || !prev_node || !prev_key || !new_node || !new_key || !gtm_index_ok(index))
    return GRACE_INVALID_ARG;
  if (B <= 0 || K <= 0 || M_prev <= 0 || prefix_len < 0 || prefix_len >= 4) return GRACE_INVALID_ARG;
  const int n = B * K;
  grace::beam_update_csr_kernel<<<(n + 255) / 256, 256, 0, (cudaStream_t)stream>>>(
      parent, token, score, prev_node, prev_key, *index, new_node, new_key, B, K, M_prev, prefix_len, d_status);
  GRACE_LAUNCH_CHECK();
  return GRACE_OK;
}
