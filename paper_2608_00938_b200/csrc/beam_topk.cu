// Beam x codebook top-k (Sections 3.1, 3.3): per request, the K best of N = M * |V| candidates
// under the total order (value descending, flat index ascending), returned in that order.
//
// The candidates are read from HBM once.  Three launches:
//   1. sample   : per request, 4096 sample points x 8 consecutive floats (one 32-byte sector per
//                 point, one point per N/4096-element stratum).  The r-th largest sample, with r
//                 a few standard deviations above K * (samples / N), becomes a threshold that
//                 with high probability has between K and `kCap` candidates above it.
//   2. collect  : the one full pass.  Every candidate above the threshold is appended to the
//                 request's list (warp-aggregated atomics; hits are a fraction of a percent).
//   3. finalize : requests whose list came out short or overflowed (and every request when N is
//                 small) are first redone by a three-level radix select that resolves ties by
//                 index (one CTA per request, exact for any input).  Then: bitonic sort of the list on (key, index), write the first K; if the threshold
//                 was -inf and fewer than K finite candidates exist, the remaining slots are the
//                 lowest-index -inf candidates.
// The result is exact whatever the threshold; the threshold only decides which path runs.
#include "common.cuh"

namespace grace {

constexpr int kCap = 8192;               // list capacity per request (entries)
constexpr int kHeaderWords = 16;         // per-request header, 64 bytes
constexpr int kSamplePoints = 4096;
constexpr int kSampleSize = kSamplePoints * 8;
constexpr int kTopkThreads = 1024;
constexpr int kMaxK = 4096;              // largest K supported
constexpr int kBucketMax = 128;          // finalize: largest bucket the counting sort ranks by comparison

struct TopkHeader {                      // lives in the workspace, one per request
  uint32_t count;                        // entries appended (may exceed kCap: overflow)
  uint32_t t_excl;                       // collect keys strictly above this
  uint32_t need_exact;
  uint32_t pad[kHeaderWords - 3];
};

__host__ __device__ inline size_t topk_header_bytes(int B) { return (size_t)B * sizeof(TopkHeader); }

// Where the candidates come from.  Dense: an array [B][N].  Masked: they are never materialised; candidate i
// of request b is token v = i % V of row r = (b * N + i) / V, worth row_score[r] + (logits[r][v] - row_lse[r])
// if bit v of the row's allow words is set and -inf otherwise: the very arithmetic of the fused mask kernel, so
// both forms select identically.  Logits are read only where a token of the four is allowed.
struct CandSrc {
  const float* data;            // dense: candidates; masked: logits [B * M][V]
  const uint64_t* allow;        // masked: [B * M][V / 64]; nullptr = dense
  const float* row_score;       // masked: [B * M]
  const float* row_lse;         // masked: [B * M]
  int64_t N;
  int V, log2_V;                // log2_V >= 0 when V is a power of two

  __device__ __forceinline__ float4 load4(int b, int64_t i4, bool streaming) const {
    if (allow == nullptr) {
      const float4* p = reinterpret_cast<const float4*>(data + (int64_t)b * N) + i4;
      return streaming ? __ldcs(p) : __ldg(p);
    }
    const int64_t g = (int64_t)b * N + i4 * 4;               // global element index; V % 64 == 0: 4 tokens of one word
    const int64_t r = (log2_V >= 0) ? (g >> log2_V) : (g / V);
    const int v = (int)(g - r * V);
    const uint32_t nib = (uint32_t)(__ldg(allow + r * (V >> 6) + (v >> 6)) >> (v & 63)) & 0xfu;
    const float ninf = __int_as_float(0xff800000);
    if (nib == 0u) return make_float4(ninf, ninf, ninf, ninf);
    const float4 x = __ldg(reinterpret_cast<const float4*>(data + g));
    const float lse = __ldg(row_lse + r), sc = __ldg(row_score + r);
    return make_float4((nib & 1u) ? sc + (x.x - lse) : ninf, (nib & 2u) ? sc + (x.y - lse) : ninf,
                       (nib & 4u) ? sc + (x.z - lse) : ninf, (nib & 8u) ? sc + (x.w - lse) : ninf);
  }
  __device__ __forceinline__ float load1(int b, int64_t i) const {
    if (allow == nullptr) return __ldg(data + (int64_t)b * N + i);
    const int64_t g = (int64_t)b * N + i;
    const int64_t r = (log2_V >= 0) ? (g >> log2_V) : (g / V);
    const int v = (int)(g - r * V);
    if (!((__ldg(allow + r * (V >> 6) + (v >> 6)) >> (v & 63)) & 1ull)) return __int_as_float(0xff800000);
    return __ldg(row_score + r) + (__ldg(data + g) - __ldg(row_lse + r));
  }
};

// ---- block primitives (kTopkThreads threads) -------------------------------------------
__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    uint32_t o = __shfl_up_sync(kFullMask, v, d);
    if (lane >= d) v += o;
  }
  return v;
}

// Exclusive prefix sum over the block; *total receives the block sum.  scratch: 33 words.
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* scratch, uint32_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t incl = warp_incl_scan(v);
  __syncthreads();                                   // scratch may still be read from a previous call
  if (lane == 31) scratch[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    uint32_t w = (lane < (int)(blockDim.x >> 5)) ? scratch[lane] : 0u;
    uint32_t wi = warp_incl_scan(w);
    scratch[lane] = wi - w;
    if (lane == 31) scratch[32] = wi;
  }
  __syncthreads();
  *total = scratch[32];
  return scratch[warp] + incl - v;
}

// One radix level.  hist[nbins] holds counts of digit values among the still-matching keys.
// Finds the digit d with (#keys with larger digit) < k <= (#keys with digit >= d); returns d and
// reduces *k by the number of keys with a larger digit.  nbins <= 4 * blockDim.x.
__device__ __forceinline__ uint32_t pick_digit(const uint32_t* hist, int nbins, uint32_t* k,
                                               uint32_t* scratch, uint32_t* result) {
  // thread t owns bins [4t, 4t+4) counted from the top: bin index nbins-1-4t-j
  uint32_t c[4];
  uint32_t mine = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int bin = nbins - 1 - (4 * (int)threadIdx.x + j);
    c[j] = (bin >= 0) ? hist[bin] : 0u;
    mine += c[j];
  }
  uint32_t total;
  uint32_t above = block_excl_scan(mine, scratch, &total);   // keys in bins above this thread's
  const uint32_t want = *k;
  __syncthreads();
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int bin = nbins - 1 - (4 * (int)threadIdx.x + j);
    if (bin >= 0 && above < want && want <= above + c[j]) {
      result[0] = (uint32_t)bin;
      result[1] = want - above;
    }
    above += c[j];
  }
  __syncthreads();
  *k = result[1];
  return result[0];
}

// ---- 1. sample -------------------------------------------------------------------------------
// Each thread reads 4 sample points (32 keys) and keeps its two largest; the threshold is at (or a few
// keys below) the r-th largest of those 2 * 1024 keys.  Dropping a thread's third-largest key can only lower the
// threshold (more candidates collected), never raise it, so the guarantee "at least K above the
// threshold with high probability" is kept while the selection works on 2048 keys instead of 32768.
__global__ void __launch_bounds__(kTopkThreads)
topk_sample_kernel(const CandSrc src, uint32_t rank, TopkHeader* hdr) {
  pdl_wait();
  pdl_trigger();
  __shared__ uint32_t hist[4096];
  __shared__ uint32_t scratch[40];
  __shared__ uint32_t result[2];
  __shared__ uint32_t red[64];
  const int b = blockIdx.x;
  const int64_t N = src.N;
  const uint32_t stratum = (uint32_t)(N / kSamplePoints) & ~7u;     // multiple of 8 elements (N < 2^31)
  const uint32_t slots = stratum >> 3;
  float4 v[2 * (kSamplePoints / kTopkThreads)];
#pragma unroll
  for (int q = 0; q < kSamplePoints / kTopkThreads; ++q) {
    const uint32_t p = q * kTopkThreads + threadIdx.x;
    uint32_t h = p * 0x9e3779b1u + (uint32_t)b * 0x85ebca77u;      // where in its stratum point p of request b lies
    h ^= h >> 16; h *= 0x85ebca6bu; h ^= h >> 13; h *= 0xc2b2ae35u; h ^= h >> 16;
    const uint32_t at4 = (p * stratum + __umulhi(h, slots) * 8u) >> 2;
    v[2 * q] = src.load4(b, at4, false);
    v[2 * q + 1] = src.load4(b, at4 + 1, false);
  }
  // the two largest of the thread's 32 values, on the floats themselves (a NaN never wins a maximum, so it
  // cannot become the threshold; the collecting pass reports it)
  float m1 = __int_as_float(0xff800000), m2 = m1;
#pragma unroll
  for (int q = 0; q < 2 * (kSamplePoints / kTopkThreads); ++q) {
    const float x[4] = {v[q].x, v[q].y, v[q].z, v[q].w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      m2 = fmaxf(m2, fminf(m1, x[j]));
      m1 = fmaxf(m1, x[j]);
    }
  }
  const uint32_t top1 = ordered_key(m1), top2 = ordered_key(m2);
  // The threshold need not be the r-th largest key itself: any value at or below it with few keys in
  // between will do.  So instead of a full radix selection, histogram the keys over 4096 equal ranges
  // between the smallest and the largest, take the lower edge of the range that holds rank r, and look
  // closer (the same again inside that range) only while the range holds more than a few keys, which
  // happens when an outlier stretches the span.
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t kmin = top2, kmax = top1;
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) {
    kmin = min(kmin, __shfl_xor_sync(kFullMask, kmin, d));
    kmax = max(kmax, __shfl_xor_sync(kFullMask, kmax, d));
  }
  if (lane == 0) { red[warp] = kmin; red[32 + warp] = kmax; }
  __syncthreads();
  kmin = red[lane];
  kmax = red[32 + lane];
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) {
    kmin = min(kmin, __shfl_xor_sync(kFullMask, kmin, d));
    kmax = max(kmax, __shfl_xor_sync(kFullMask, kmax, d));
  }
  uint32_t k = rank, lo = kmin, span = kmax - kmin, prefix = kmin;
#pragma unroll 1
  for (int level = 0; level < 4; ++level) {
    const int sh = max(0, 20 - __clz(span));                 // span >> sh < 4096
    for (int i = threadIdx.x; i < 4096; i += kTopkThreads) hist[i] = 0;
    __syncthreads();
    if (top1 - lo <= span) atomicAdd(&hist[(top1 - lo) >> sh], 1u);
    if (top2 - lo <= span) atomicAdd(&hist[(top2 - lo) >> sh], 1u);
    __syncthreads();
    const uint32_t d = pick_digit(hist, 4096, &k, scratch, result);
    const uint32_t in_range = hist[d];
    prefix = lo + (d << sh);                                 // at least `rank` keys are >= prefix
    if (sh == 0 || in_range <= 4u) break;
    lo = prefix;
    span = (1u << sh) - 1u;
  }
  if (threadIdx.x == 0) {
    hdr[b].count = 0;
    hdr[b].need_exact = 0;
    hdr[b].t_excl = (prefix <= kKeyNegInf) ? kKeyNegInf : prefix - 1;
  }
}

__global__ void topk_reset_kernel(TopkHeader* hdr, int B) {
  pdl_wait();
  pdl_trigger();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < B) { hdr[b].count = 0; hdr[b].t_excl = 0; hdr[b].need_exact = 1; }
}

// ---- 2. collect ------------------------------------------------------------------------------
constexpr int kCollectThreads = 256;
constexpr int kCollectUnroll = 8;                         // float4 loads in flight per thread
constexpr int kCollectWarps = kCollectThreads / 32;

constexpr int kWarpStage = 256;                           // hits staged per warp before a flush (dense pass)

// Appends the warp's staged hits to the request's list with one global atomic; returns true once the list
// has overflowed (the exact path will redo the request, so the caller may stop scanning).
__device__ __forceinline__ bool warp_flush(uint2* wstage, uint32_t* wcount, uint32_t* list_count, uint2* list) {
  __syncwarp();
  const int lane = threadIdx.x & 31;
  const uint32_t n = *reinterpret_cast<volatile uint32_t*>(wcount);
  if (n == 0) return false;
  uint32_t dst = 0;
  if (lane == 0) dst = atomicAdd(list_count, n);
  dst = __shfl_sync(kFullMask, dst, 0);
  for (uint32_t e = lane; e < n; e += 32)
    if (dst + e < (uint32_t)kCap) list[dst + e] = wstage[e];
  __syncwarp();
  if (lane == 0) *reinterpret_cast<volatile uint32_t*>(wcount) = 0;
  __syncwarp();
  return dst + n > (uint32_t)kCap;
}

// One float4 of candidates with at least one lane of the warp above the threshold (entered warp-uniformly).
__device__ __forceinline__ bool collect_hits(const float4 v, bool mine, uint32_t i4, float thr, uint2* wstage,
                                             uint32_t* wcount, uint32_t* list_count, uint2* list, bool* saw_nan) {
  bool dead = false;
  if (*reinterpret_cast<volatile uint32_t*>(wcount) > (uint32_t)(kWarpStage - 128))
    dead = warp_flush(wstage, wcount, list_count, list);
  if (mine) {
    const float x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (!(x[j] <= thr)) {
        if (x[j] != x[j]) { *saw_nan = true; continue; }
        const uint32_t pos = atomicAdd(wcount, 1u);
        wstage[pos] = make_uint2(ordered_key(x[j]), i4 * 4u + (uint32_t)j);
      }
    }
  }
  __syncwarp();
  return dead;
}

__global__ void __launch_bounds__(kCollectThreads, 5)
topk_collect_kernel(const CandSrc src, TopkHeader* hdr, uint2* lists, int32_t* d_status) {
  // grid (x, B): the CTAs of column b split request b's candidates into contiguous, equal chunks of whole
  // 256-float4 rows.  Hits are a fraction of a percent; each warp stages its own in shared memory (a
  // shared-memory atomic per hit, no scan) and appends them to the request's list with ONE global atomic
  // per flush, so the loop has no block-wide barrier and the per-request counter sees a few hundred atomics.
  __shared__ uint2 stage[kCollectWarps][kWarpStage];
  __shared__ uint32_t stage_count[kCollectWarps];
  const int b = blockIdx.y;
  const int warp = threadIdx.x >> 5;
  uint2* wstage = stage[warp];
  uint32_t* wcount = &stage_count[warp];
  if ((threadIdx.x & 31) == 0) *wcount = 0;
  __syncwarp();
  const uint32_t n4 = (uint32_t)(src.N >> 2);
  const float4* row = reinterpret_cast<const float4*>(src.data + (int64_t)b * src.N);
  uint2* list = lists + (int64_t)b * kCap;
  uint32_t* list_count = &hdr[b].count;
  const uint32_t rows_total = (n4 + kCollectThreads - 1) / kCollectThreads;
  const uint32_t rows_per_cta = (rows_total + gridDim.x - 1) / gridDim.x;
  uint32_t r = blockIdx.x * rows_per_cta;
  const uint32_t r_end = min(rows_total, r + rows_per_cta);
  const uint32_t r_full = min(r_end, n4 / kCollectThreads);      // rows below this one are wholly in bounds
  const float ninf = __int_as_float(0xff800000);
  // This kernel is scheduled while the sampling kernel still runs, and only the threshold depends on that
  // kernel: the candidates were complete before it started (it waits for its own predecessors before it
  // lets this kernel be scheduled).  So the first tile of the chunk is requested now, past the L1 (which
  // may hold lines of an earlier call's candidates), and the memory system works under the sampling
  // kernel instead of idling.  (Fetching further rows into shared memory at this point was measured
  // slower: the shared-memory carve-out it needs shrinks the L1 the streaming loads pass through.)
  const uint32_t i_first = r * kCollectThreads + threadIdx.x;
  float4 v[kCollectUnroll];
#pragma unroll
  for (int u = 0; u < kCollectUnroll; ++u)
    v[u] = (r + u < r_full) ? __ldcg(row + i_first + u * kCollectThreads) : make_float4(ninf, ninf, ninf, ninf);
  pdl_wait();
  pdl_trigger();
  const uint32_t t_excl = __ldcg(&hdr[b].t_excl);
  // the same threshold as a float: key(x) > t_excl  <=>  x > thr for every non-NaN x
  const float thr = __uint_as_float((t_excl & 0x80000000u) ? (t_excl ^ 0x80000000u) : ~t_excl);
  bool saw_nan = false, dead = false;
#pragma unroll
  for (int u = 0; u < kCollectUnroll; ++u) {
    // !(x <= thr): above the threshold, or NaN
    const bool mine = !(v[u].x <= thr) || !(v[u].y <= thr) || !(v[u].z <= thr) || !(v[u].w <= thr);
    if (__any_sync(kFullMask, mine))
      dead |= collect_hits(v[u], mine, i_first + u * kCollectThreads, thr, wstage, wcount, list_count, list, &saw_nan);
  }
  if (r < r_full) r = min(r + kCollectUnroll, r_full);
  for (; r + kCollectUnroll <= r_full && !dead; r += kCollectUnroll) {
    const uint32_t i0 = r * kCollectThreads + threadIdx.x;
#pragma unroll
    for (int u = 0; u < kCollectUnroll; ++u) v[u] = __ldcs(row + i0 + u * kCollectThreads);
#pragma unroll
    for (int u = 0; u < kCollectUnroll; ++u) {
      const bool mine = !(v[u].x <= thr) || !(v[u].y <= thr) || !(v[u].z <= thr) || !(v[u].w <= thr);
      if (__any_sync(kFullMask, mine))
        dead |= collect_hits(v[u], mine, i0 + u * kCollectThreads, thr, wstage, wcount, list_count, list, &saw_nan);
    }
  }
  for (; r < r_end && !dead; ++r) {
    const uint32_t i = r * kCollectThreads + threadIdx.x;
    const float4 x = (i < n4) ? __ldcs(row + i) : make_float4(ninf, ninf, ninf, ninf);
    const bool mine = !(x.x <= thr) || !(x.y <= thr) || !(x.z <= thr) || !(x.w <= thr);
    if (__any_sync(kFullMask, mine))
      dead |= collect_hits(x, mine, i, thr, wstage, wcount, list_count, list, &saw_nan);
  }
  warp_flush(wstage, wcount, list_count, list);
  if (saw_nan) flag_status(d_status, GRACE_DEV_NAN);
}

// Collecting pass over candidates that are not materialised: the unit of work is one 64-bit allow word (64
// tokens of one row).  A zero word costs one 8-byte load; otherwise the thread walks the word's set bits four at a
// time: the four logits are requested together, then tested (work follows the allowed tokens, not the codebook:
// a pass over 16-byte groups of four tokens spent most of its instructions on tokens that were not allowed).
// Hits are rare and go to the warp's own staging list, as in the dense pass (a full stage: straight to the
// request's list); no block-wide barrier in the loop.
constexpr int kCollectWords = 8;                          // allow words in flight per thread

__global__ void __launch_bounds__(kCollectThreads, 4)
topk_collect_masked_kernel(const CandSrc src, TopkHeader* hdr, uint2* lists, int32_t* d_status) {
  pdl_wait();
  pdl_trigger();
  __shared__ uint2 stage[kCollectWarps][kWarpStage];
  __shared__ uint32_t stage_count[kCollectWarps];
  const int b = blockIdx.y;
  const int warp = threadIdx.x >> 5;
  uint2* wstage = stage[warp];
  uint32_t* wcount = &stage_count[warp];
  if ((threadIdx.x & 31) == 0) *wcount = 0;
  __syncwarp();
  const uint32_t n_words = (uint32_t)(src.N >> 6);
  const uint64_t* words = src.allow + (((int64_t)b * src.N) >> 6);
  uint2* list = lists + (int64_t)b * kCap;
  uint32_t* list_count = &hdr[b].count;
  const uint32_t rows_total = (n_words + kCollectThreads - 1) / kCollectThreads;      // rows of 256 words
  const uint32_t rows_per_cta = (rows_total + gridDim.x - 1) / gridDim.x;
  const uint32_t r_begin = blockIdx.x * rows_per_cta;
  const uint32_t r_end = min(rows_total, r_begin + rows_per_cta);
  const uint32_t t_excl = __ldcg(&hdr[b].t_excl);
  const float thr = __uint_as_float((t_excl & 0x80000000u) ? (t_excl ^ 0x80000000u) : ~t_excl);
  bool saw_nan = false, dead = false;
  for (uint32_t r0 = r_begin; r0 < r_end && !dead; r0 += kCollectWords) {
    uint64_t w[kCollectWords];
#pragma unroll
    for (int u = 0; u < kCollectWords; ++u) {
      const uint32_t i = (r0 + u) * kCollectThreads + threadIdx.x;
      w[u] = (r0 + u < r_end && i < n_words) ? __ldcs(words + i) : 0ull;
    }
#pragma unroll 1
    for (int u = 0; u < kCollectWords; ++u) {
      const uint64_t bits = w[u];
      if (bits == 0ull) continue;
      const uint32_t i = (r0 + u) * kCollectThreads + threadIdx.x;
      const int64_t g0 = (int64_t)b * src.N + ((int64_t)i << 6);    // first token of the word, global element index
      const int64_t r = (src.log2_V >= 0) ? (g0 >> src.log2_V) : (g0 / src.V);
      const float lse = __ldg(src.row_lse + r), sc = __ldg(src.row_score + r);
      const float* tok = src.data + g0;
      uint64_t rest = bits;
#pragma unroll 1
      while (rest != 0ull) {
        // the next (up to) four allowed tokens of the word: their logits are requested together
        int pos[4];
        float x[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          pos[e] = (rest != 0ull) ? __ffsll((long long)rest) - 1 : -1;
          rest &= rest - 1ull;
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) x[e] = (pos[e] >= 0) ? __ldg(tok + pos[e]) : 0.f;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (pos[e] < 0) continue;
          const float val = sc + (x[e] - lse);
          if (val <= thr) continue;                               // NaN falls through
          if (val != val) { saw_nan = true; continue; }
          const uint2 entry = make_uint2(ordered_key(val), (i << 6) + (uint32_t)pos[e]);
          const uint32_t at = atomicAdd(wcount, 1u);
          if (at < (uint32_t)kWarpStage) {
            wstage[at] = entry;
          } else {                                                // stage full: straight to the request's list
            const uint32_t gpos = atomicAdd(list_count, 1u);
            if (gpos < (uint32_t)kCap) list[gpos] = entry;
          }
        }
      }
    }
    __syncwarp();
    const uint32_t staged = *reinterpret_cast<volatile uint32_t*>(wcount);
    if (staged >= (uint32_t)kWarpStage / 2) {                     // uniform over the warp
      if (staged > (uint32_t)kWarpStage) {                        // the overhang went to the list already
        __syncwarp();
        if ((threadIdx.x & 31) == 0) *reinterpret_cast<volatile uint32_t*>(wcount) = (uint32_t)kWarpStage;
      }
      dead = warp_flush(wstage, wcount, list_count, list);
    }
  }
  {
    __syncwarp();
    const uint32_t staged = *reinterpret_cast<volatile uint32_t*>(wcount);
    if (staged > (uint32_t)kWarpStage) {
      __syncwarp();
      if ((threadIdx.x & 31) == 0) *reinterpret_cast<volatile uint32_t*>(wcount) = (uint32_t)kWarpStage;
    }
    warp_flush(wstage, wcount, list_count, list);
  }
  if (saw_nan) flag_status(d_status, GRACE_DEV_NAN);
}

// ---- 3. exact --------------------------------------------------------------------------------
// One CTA per request.  Three histogram passes over the row fix the K-th key exactly; a fourth
// pass in index order writes the keys above it and the first ties.
__device__ void topk_exact_select(const CandSrc& src, int K, uint2* lists, int b,
                                  uint32_t* hist /*4096*/, uint32_t* scratch /*40*/, uint32_t* result /*2*/,
                                  int32_t* d_status) {
  const int64_t n4 = src.N >> 2;
  uint32_t k = (uint32_t)K, prefix = 0;
  const int shifts[3] = {20, 8, 0};
  const int bits[3] = {12, 12, 8};
  bool saw_nan = false;
#pragma unroll 1
  for (int level = 0; level < 3; ++level) {
    const int nb = 1 << bits[level];
    for (int i = threadIdx.x; i < 4096; i += kTopkThreads) hist[i] = 0;
    __syncthreads();
    const int hi_shift = shifts[level] + bits[level];
    uint32_t n_ninf = 0;            // -inf dominates masked rows: count it in a register
    for (int64_t i = threadIdx.x; i < n4; i += kTopkThreads) {
      const float4 v = src.load4(b, i, false);
      const float x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (level == 0 && x[j] != x[j]) saw_nan = true;
        const uint32_t u = ordered_key(x[j]);
        if (u == kKeyNegInf) { ++n_ninf; continue; }
        const bool match = (level == 0) || ((u >> hi_shift) == prefix);
        if (match) atomicAdd(&hist[(u >> shifts[level]) & (nb - 1)], 1u);
      }
    }
    if (n_ninf != 0 && ((level == 0) || ((kKeyNegInf >> hi_shift) == prefix)))
      atomicAdd(&hist[(kKeyNegInf >> shifts[level]) & (nb - 1)], n_ninf);
    __syncthreads();
    const uint32_t d = pick_digit(hist, nb, &k, scratch, result);
    prefix = (prefix << bits[level]) | d;
  }
  if (saw_nan) flag_status(d_status, GRACE_DEV_NAN);
  // prefix = exact K-th key; k = number of ties (key == prefix) to take, lowest indices first
  const uint32_t kth = prefix, n_ties = k, n_above = (uint32_t)K - k;
  uint2* list = lists + (int64_t)b * kCap;
  uint32_t done_above = 0, done_ties = 0;
  for (int64_t base = 0; base < n4; base += kTopkThreads) {
    const int64_t i = base + threadIdx.x;
    float4 v = make_float4(0, 0, 0, 0);
    uint32_t key[4] = {0, 0, 0, 0};
    uint32_t above = 0, ties = 0;
    if (i < n4) {
      v = src.load4(b, i, false);
      key[0] = ordered_key(v.x); key[1] = ordered_key(v.y); key[2] = ordered_key(v.z); key[3] = ordered_key(v.w);
#pragma unroll
      for (int j = 0; j < 4; ++j) { above += key[j] > kth; ties += key[j] == kth; }
    }
    uint32_t tot_above, tot_ties;
    uint32_t pa = block_excl_scan(above, scratch, &tot_above) + done_above;
    uint32_t pt = block_excl_scan(ties, scratch, &tot_ties) + done_ties;
    if (i < n4) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (key[j] > kth) {
          if (pa < n_above) list[pa] = make_uint2(key[j], (uint32_t)(i * 4 + j));
          ++pa;
        } else if (key[j] == kth) {
          if (pt < n_ties) list[n_above + pt] = make_uint2(key[j], (uint32_t)(i * 4 + j));
          ++pt;
        }
      }
    }
    done_above += tot_above;
    done_ties += tot_ties;
    if (done_ties >= n_ties && done_above >= n_above) break;   // uniform across the block
  }
  __syncthreads();
}

// ---- 4. finalize -----------------------------------------------------------------------------
// Descending bitonic sort of n = 1024 * E keys (E = 1, 2, 4, 8 per thread).  Thread t owns the E
// consecutive keys t*E..t*E+E-1 in registers and a warp owns 32*E consecutive keys, so every
// compare-exchange with stride < 32*E is a register swap or a warp shuffle; only the strides
// >= 32*E go through shared memory with a block-wide barrier.
template <int E>
__device__ __forceinline__ void bitonic_regs(unsigned long long (&v)[E], uint32_t base_index, uint32_t size,
                                             uint32_t first_stride) {
  // compare-exchange steps of one merge phase (`size`) for strides first_stride .. 1, all < 32*E
  for (uint32_t stride = first_stride; stride >= (uint32_t)E; stride >>= 1) {
    const uint32_t lane_xor = stride / E;
#pragma unroll
    for (int e = 0; e < E; ++e) {
      const uint32_t i = base_index + e;
      const unsigned long long other = __shfl_xor_sync(kFullMask, v[e], lane_xor);
      const bool desc = (i & size) == 0;
      const bool lower = (i & stride) == 0;
      const bool keep_max = (desc == lower);
      v[e] = keep_max ? (v[e] > other ? v[e] : other) : (v[e] < other ? v[e] : other);
    }
    if (stride == 1) break;
  }
#pragma unroll
  for (int st = E / 2; st >= 1; st >>= 1) {
    if ((uint32_t)st > first_stride) continue;
#pragma unroll
    for (int e = 0; e < E; ++e) {
      if ((e & st) == 0) {
        const uint32_t i = base_index + e;
        const bool desc = (i & size) == 0;
        const unsigned long long a = v[e], c = v[e + st];
        const bool swap = desc ? (a < c) : (a > c);
        if (swap) { v[e] = c; v[e + st] = a; }
      }
    }
  }
}

template <int E>
__device__ void block_bitonic_sort_desc(unsigned long long* keys) {
  constexpr uint32_t n = 1024u * E;
  constexpr uint32_t warp_span = 32u * E;
  const uint32_t base_index = threadIdx.x * E;
  unsigned long long v[E];
#pragma unroll
  for (int e = 0; e < E; ++e) v[e] = keys[base_index + e];
  // phases whose every stride stays inside a warp
  for (uint32_t size = 2; size <= warp_span && size <= n; size <<= 1) bitonic_regs<E>(v, base_index, size, size >> 1);
  for (uint32_t size = warp_span << 1; size <= n; size <<= 1) {
#pragma unroll
    for (int e = 0; e < E; ++e) keys[base_index + e] = v[e];
    __syncthreads();
    for (uint32_t stride = size >> 1; stride >= warp_span; stride >>= 1) {
      for (uint32_t t = threadIdx.x; t < (n >> 1); t += kTopkThreads) {
        const uint32_t lo = 2 * t - (t & (stride - 1));
        const uint32_t hi = lo + stride;
        const bool desc = ((lo & size) == 0);
        const unsigned long long a = keys[lo], d = keys[hi];
        if ((a < d) == desc) { keys[lo] = d; keys[hi] = a; }
      }
      __syncthreads();
    }
#pragma unroll
    for (int e = 0; e < E; ++e) v[e] = keys[base_index + e];
    bitonic_regs<E>(v, base_index, size, warp_span >> 1);
  }
#pragma unroll
  for (int e = 0; e < E; ++e) keys[base_index + e] = v[e];
  __syncthreads();
}

__global__ void __launch_bounds__(kTopkThreads)
topk_finalize_kernel(const CandSrc src, int K, int K_out, int V, TopkHeader* hdr,
                     uint2* lists, int force_exact, float* out_score, int32_t* out_flat, int32_t* out_parent,
                     int32_t* out_token, int32_t* d_status) {
  // K = min(requested, N) entries are selected; rows of the outputs are K_out = requested wide.
  pdl_wait();
  pdl_trigger();
  extern __shared__ unsigned long long sort_keys_raw[];     // kCap + kMaxK keys, then a 4096-bin histogram
  unsigned long long* sort_keys = sort_keys_raw;
  __shared__ uint32_t scratch[40];
  __shared__ uint32_t result[2];
  __shared__ uint32_t red[64];
  const int b = blockIdx.x;
  uint32_t c = hdr[b].count;
  // Exact multi-pass selection when the sampled threshold did not deliver (list short although the
  // threshold was not -inf, or list overflow) and for shapes that skip sampling altogether.
  const bool need_exact = force_exact || c > (uint32_t)kCap || (c < (uint32_t)K && hdr[b].t_excl != kKeyNegInf);
  if (need_exact) {
    if (!force_exact && threadIdx.x == 0) flag_status(d_status, GRACE_DEV_TOPK_EXACT_PATH);
    topk_exact_select(src, K, lists, b, reinterpret_cast<uint32_t*>(sort_keys), scratch, result, d_status);
    __syncthreads();
    c = (uint32_t)K;
  }
  c = min(c, (uint32_t)kCap);
  const uint2* list = lists + (int64_t)b * kCap;
  unsigned long long* all_keys = sort_keys;                 // c composite keys (value key, ~index)
  unsigned long long* top_keys = sort_keys + kCap;          // the K winners (fast path: plus one bucket's overhang)
  uint32_t* hist = reinterpret_cast<uint32_t*>(top_keys + kMaxK + kBucketMax);
  uint32_t* offs = hist + 4096;
  const int64_t N = src.N;
  const uint32_t n_out = min(c, (uint32_t)K);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t kmin = 0xffffffffu, kmax = 0u;
  for (uint32_t i = threadIdx.x; i < c; i += kTopkThreads) {
    const uint2 e = list[i];
    all_keys[i] = ((unsigned long long)e.x << 32) | (unsigned long long)(0xffffffffu - e.y);
    kmin = min(kmin, e.x);
    kmax = max(kmax, e.x);
  }
  for (int i = threadIdx.x; i < 4096; i += kTopkThreads) hist[i] = 0;
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) {
    kmin = min(kmin, __shfl_xor_sync(kFullMask, kmin, d));
    kmax = max(kmax, __shfl_xor_sync(kFullMask, kmax, d));
  }
  if (lane == 0) { red[warp] = kmin; red[32 + warp] = kmax; }
  __syncthreads();
  kmin = red[lane];
  kmax = red[32 + lane];
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) {
    kmin = min(kmin, __shfl_xor_sync(kFullMask, kmin, d));
    kmax = max(kmax, __shfl_xor_sync(kFullMask, kmax, d));
  }
  // Fast path: a counting sort.  The value keys are spread over up to 4096 buckets by a monotone map
  // (equal-width ranges of the key between the smallest and largest collected key), a scan from the top
  // gives every bucket its first rank, the buckets that start below rank K are scattered to their rank
  // ranges, and a key's rank is its bucket's first rank plus the keys of the same bucket that beat it
  // under the total order.  Buckets hold a handful of keys unless the keys are clustered or tied in
  // thousands; then the radix selection and bitonic sort below do the job.
  bool fast = (c != 0);
  if (fast) {
    const uint32_t span = kmax - kmin;
    const int sh = max(0, 20 - __clz(span));                // span >> sh < 4096
    for (uint32_t i = threadIdx.x; i < c; i += kTopkThreads)
      atomicAdd(&hist[((uint32_t)(all_keys[i] >> 32) - kmin) >> sh], 1u);
    __syncthreads();
    uint32_t c4[4];
    uint32_t mine = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      c4[j] = hist[4095 - (4 * (int)threadIdx.x + j)];
      mine += c4[j];
    }
    uint32_t total;
    uint32_t above = block_excl_scan(mine, scratch, &total);
    bool big = false;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int bin = 4095 - (4 * (int)threadIdx.x + j);
      offs[bin] = above;
      if (above < n_out) {
        if (c4[j] > (uint32_t)kBucketMax) big = true;
        if (n_out <= above + c4[j]) result[0] = above + c4[j];   // keys in the buckets that start below rank K
      }
      above += c4[j];
    }
    fast = (__syncthreads_or(big ? 1 : 0) == 0);
    if (fast) {
      for (uint32_t i = threadIdx.x; i < c; i += kTopkThreads) {
        const unsigned long long u = all_keys[i];
        const uint32_t bk = ((uint32_t)(u >> 32) - kmin) >> sh;
        const uint32_t first = offs[bk];
        if (first < n_out) top_keys[first + atomicSub(&hist[bk], 1u) - 1u] = u;
      }
      __syncthreads();
      const uint32_t n_placed = result[0];
      for (uint32_t p = threadIdx.x; p < n_placed; p += kTopkThreads) {
        const unsigned long long u = top_keys[p];
        const uint32_t key = (uint32_t)(u >> 32);
        const uint32_t bk = (key - kmin) >> sh;
        const uint32_t first = offs[bk];
        const uint32_t last = (bk != 0) ? offs[bk - 1] : c;   // the next lower bucket starts where this one ends
        uint32_t rank = first;
        for (uint32_t q = first; q < last; ++q) rank += (top_keys[q] > u) ? 1u : 0u;
        if (rank < n_out) {
          uint32_t idx = 0xffffffffu - (uint32_t)(u & 0xffffffffull);
          if ((int64_t)idx >= N) { flag_status(d_status, GRACE_DEV_BAD_INDEX); idx = 0; }    // cannot happen; never fault
          const int64_t o = (int64_t)b * K_out + rank;
          // the key maps back to the candidate's own bits, except that it does not tell -0 from +0
          out_score[o] = (key == 0x80000000u) ? src.load1(b, idx)
                                              : __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
          if (out_flat) out_flat[o] = (int32_t)idx;
          if (out_parent) out_parent[o] = (int32_t)(idx / (uint32_t)V);
          if (out_token) out_token[o] = (int32_t)(idx % (uint32_t)V);
        }
      }
    } else {
      for (int i = threadIdx.x; i < 4096; i += kTopkThreads) hist[i] = 0;
    }
  }
  __syncthreads();
  if (!fast && c != 0) {
    unsigned long long* to_sort = all_keys;
    uint32_t n_keep = c;
    if (c > (uint32_t)K) {
      // Composite keys are distinct, so the K-th largest is well defined: six radix levels over
      // the 64 bits (value key first, then the index part that breaks ties towards low indices).
      uint32_t k = (uint32_t)K;
      unsigned long long prefix = 0ull;
      const int shifts[6] = {52, 40, 32, 20, 8, 0};
      const int bits[6] = {12, 12, 8, 12, 12, 8};
  #pragma unroll 1
      for (int level = 0; level < 6; ++level) {
        const int nb = 1 << bits[level];
        for (int i = threadIdx.x; i < 4096; i += kTopkThreads) hist[i] = 0;
        __syncthreads();
        const int hi_shift = shifts[level] + bits[level];
        for (uint32_t i = threadIdx.x; i < c; i += kTopkThreads) {
          const unsigned long long u = all_keys[i];
          const bool match = (level == 0) || ((u >> hi_shift) == prefix);
          if (match) atomicAdd(&hist[(uint32_t)(u >> shifts[level]) & (nb - 1)], 1u);
        }
        __syncthreads();
        const uint32_t d = pick_digit(hist, nb, &k, scratch, result);
        prefix = (prefix << bits[level]) | (unsigned long long)d;
      }
      const unsigned long long kth = prefix;                  // exactly K keys are >= kth
      uint32_t done = 0;
      for (uint32_t base = 0; base < c; base += kTopkThreads) {
        const uint32_t i = base + threadIdx.x;
        const unsigned long long u = (i < c) ? all_keys[i] : 0ull;
        const bool win = (i < c) && (u >= kth);
        uint32_t total;
        const uint32_t pos = block_excl_scan(win ? 1u : 0u, scratch, &total) + done;
        if (win) top_keys[pos] = u;
        done += total;
      }
      to_sort = top_keys;
      n_keep = (uint32_t)K;
    }
    uint32_t n_sort = 1024;
    while (n_sort < n_keep) n_sort <<= 1;
    __syncthreads();
    for (uint32_t i = n_keep + threadIdx.x; i < n_sort; i += kTopkThreads) to_sort[i] = 0ull;
    __syncthreads();
    switch (n_sort) {
      case 1024: block_bitonic_sort_desc<1>(to_sort); break;
      case 2048: block_bitonic_sort_desc<2>(to_sort); break;
      case 4096: block_bitonic_sort_desc<4>(to_sort); break;
      default: block_bitonic_sort_desc<8>(to_sort); break;
    }
    sort_keys = to_sort;
    for (uint32_t i = threadIdx.x; i < n_out; i += kTopkThreads) {
      uint32_t idx = 0xffffffffu - (uint32_t)(sort_keys[i] & 0xffffffffull);
      if ((int64_t)idx >= N) { flag_status(d_status, GRACE_DEV_BAD_INDEX); idx = 0; }    // cannot happen; never fault
      const int64_t o = (int64_t)b * K_out + i;
      out_score[o] = src.load1(b, idx);
      if (out_flat) out_flat[o] = (int32_t)idx;
      if (out_parent) out_parent[o] = (int32_t)(idx / (uint32_t)V);
      if (out_token) out_token[o] = (int32_t)(idx % (uint32_t)V);
    }
  }
  if (c < (uint32_t)K) {
    // Threshold was -inf and the row has fewer than K candidates above it: the rest of the beam
    // is the lowest-index candidates at -inf.  At most c of the first K positions are finite, so
    // scanning K positions is enough.
    const uint32_t need = (uint32_t)K - c;
    uint32_t done = 0;
    for (uint32_t base = 0; base < (uint32_t)K && done < need; base += kTopkThreads) {
      const uint32_t i = base + threadIdx.x;
      const float xi = (i < (uint32_t)K) ? src.load1(b, i) : 0.f;
      const bool is_low = (i < (uint32_t)K) && (ordered_key(xi) <= kKeyNegInf);
      uint32_t total;
      const uint32_t rank = block_excl_scan(is_low ? 1u : 0u, scratch, &total) + done;
      if (is_low && rank < need) {
        const int64_t o = (int64_t)b * K_out + c + rank;
        out_score[o] = xi;
        if (out_flat) out_flat[o] = (int32_t)i;
        if (out_parent) out_parent[o] = (int32_t)(i / (uint32_t)V);
        if (out_token) out_token[o] = (int32_t)(i % (uint32_t)V);
      }
      done += total;
    }
  }
  // A beam wider than the candidate set (K_out > N): the rest are dead beams, score -inf on candidate 0.
  for (int i = K + (int)threadIdx.x; i < K_out; i += kTopkThreads) {
    const int64_t o = (int64_t)b * K_out + i;
    out_score[o] = __int_as_float(0xff800000);
    if (out_flat) out_flat[o] = 0;
    if (out_parent) out_parent[o] = 0;
    if (out_token) out_token[o] = 0;
  }
}

// Sampling plan: rank r of the sample whose value is the threshold, or 0 if sampling is not
// worthwhile / not safe for this shape (then the exact path handles every request).
static uint32_t sample_rank(int64_t N, int K) {
  if (N < (int64_t)kSampleSize * 8 || (N & 7)) return 0;
  const double frac = (double)kSampleSize / (double)N;
  const double expect = K * frac;
  const double r = ceil(expect + 4.0 * sqrt(expect) + 8.0);
  if (r / frac > 0.75 * kCap || r > kSampleSize / 4) return 0;
  return (uint32_t)r;
}

}  // namespace grace

extern "C" size_t grace_beam_topk_workspace_bytes(int B, int64_t N, int K) {
  (void)N; (void)K;
  if (B <= 0) return 0;
  return grace::topk_header_bytes(B) + (size_t)B * grace::kCap * sizeof(uint2);
}

namespace grace {
// Shared by the public entry point and the variant that owns its scratch.
grace_status_t launch_beam_topk(const CandSrc& src_in, int B, int K, int V, float* out_score,
                                int32_t* out_flat, int32_t* out_parent, int32_t* out_token,
                                void* ws, int32_t* d_status, cudaStream_t s) {
  CandSrc src = src_in;
  const int64_t N = src.N;
  TopkHeader* hdr = reinterpret_cast<TopkHeader*>(ws);
  uint2* lists = reinterpret_cast<uint2*>(reinterpret_cast<char*>(ws) + topk_header_bytes(B));
  const int K_out = K;
  if ((int64_t)K > N) K = (int)N;                            // every candidate is selected, the rest is padding
  const uint32_t rank = sample_rank(N, K);
  static unsigned long long attrs_set_devices = 0;
  const size_t final_smem = (size_t)(kCap + kMaxK + kBucketMax) * sizeof(unsigned long long) + 2 * 4096 * sizeof(uint32_t);
  static int collect_grid_of[kMaxDevices] = {0};
  static int collect_masked_grid_of[kMaxDevices] = {0};
  DeviceSetup su(&attrs_set_devices);
  if (su) {
    GRACE_CUDA_TRY(cudaFuncSetAttribute(topk_finalize_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)final_smem));
    int n_sm = 0, per_sm = 0;
    GRACE_CUDA_TRY(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, su.dev));
    GRACE_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, topk_collect_kernel, kCollectThreads, 0));
    collect_grid_of[su.dev] = n_sm * (per_sm > 0 ? per_sm : 1);
    GRACE_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, topk_collect_masked_kernel, kCollectThreads, 0));
    collect_masked_grid_of[su.dev] = n_sm * (per_sm > 0 ? per_sm : 1);
    su.done();
  }
  const int collect_grid = collect_grid_of[su.dev];
  int force_exact = 1;
  if (rank != 0) {
    launch_pdl(topk_sample_kernel, dim3(B), dim3(kTopkThreads), 0, s, src, rank, hdr);
    GRACE_LAUNCH_CHECK();
    const int64_t tile = (int64_t)kCollectThreads * kCollectUnroll;
    const int64_t tiles_per_request = ((N >> 2) + tile - 1) / tile;
    int64_t per_request = collect_grid / B;                 // one resident wave over all requests
    if (per_request < 1) per_request = 1;
    if (per_request > tiles_per_request) per_request = tiles_per_request;
    if (src.allow != nullptr) {                              // masked: the tile is 256 x 8 allow words
      const int64_t wtile = (int64_t)kCollectThreads * kCollectWords;
      const int64_t wtiles = ((N >> 6) + wtile - 1) / wtile;
      per_request = collect_masked_grid_of[su.dev] / B;
      if (per_request < 1) per_request = 1;
      if (per_request > wtiles) per_request = wtiles;
      launch_pdl(topk_collect_masked_kernel, dim3((unsigned)per_request, (unsigned)B), dim3(kCollectThreads), 0, s, src, hdr,
                 lists, d_status);
      GRACE_LAUNCH_CHECK();
    } else {
      dim3 grid((unsigned)per_request, (unsigned)B);
      launch_pdl(topk_collect_kernel, dim3(grid), dim3(kCollectThreads), 0, s, src, hdr, lists, d_status);
      GRACE_LAUNCH_CHECK();
    }
    force_exact = 0;
  } else {
    launch_pdl(topk_reset_kernel, dim3((B + 255) / 256), dim3(256), 0, s, hdr, B);
    GRACE_LAUNCH_CHECK();
  }
  launch_pdl(topk_finalize_kernel, dim3(B), dim3(kTopkThreads), final_smem, s, src, K, K_out, V, hdr, lists, force_exact, out_score, out_flat,
                                                          out_parent, out_token, d_status);
  GRACE_LAUNCH_CHECK();
  return GRACE_OK;
}
}  // namespace grace

extern "C" grace_status_t grace_beam_topk(const float* cand, int B, int64_t N, int K, int V,
                                          float* out_score, int32_t* out_flat, int32_t* out_parent,
                                          int32_t* out_token, void* ws, size_t ws_bytes,
                                          int32_t* d_status, void* stream) {
  if (!cand || !out_score || !ws) return GRACE_INVALID_ARG;
  if (B <= 0 || N <= 0 || N >= (1ll << 31) || K < 1 || V <= 0) return GRACE_INVALID_ARG;
  if (K > 4096 || (N & 3)) return GRACE_UNSUPPORTED_SHAPE;
  if (!grace_aligned16(cand) || (reinterpret_cast<uintptr_t>(ws) & 255u)) return GRACE_INVALID_ARG;
  if (ws_bytes < grace_beam_topk_workspace_bytes(B, N, K)) return GRACE_WORKSPACE_TOO_SMALL;
  grace::CandSrc src = {cand, nullptr, nullptr, nullptr, N, V, -1};
  return grace::launch_beam_topk(src, B, K, V, out_score, out_flat, out_parent, out_token, ws,
                                 d_status, (cudaStream_t)stream);
}

extern "C" grace_status_t grace_beam_topk_masked(const float* logits, const uint64_t* allow_bits,
                                                 const float* row_score, const float* row_lse, int B, int M, int V,
                                                 int K, float* out_score, int32_t* out_flat, int32_t* out_parent,
                                                 int32_t* out_token, void* ws, size_t ws_bytes, int32_t* d_status,
                                                 void* stream) {
  if (!logits || !allow_bits || !row_score || !row_lse || !out_score || !ws) return GRACE_INVALID_ARG;
  if (B <= 0 || M <= 0 || V <= 0 || (V & 63) || K < 1) return GRACE_INVALID_ARG;
  const int64_t N = (int64_t)M * V;
  if (N >= (1ll << 31) || (int64_t)B * N >= (1ll << 40)) return GRACE_INVALID_ARG;
  if (K > 4096) return GRACE_UNSUPPORTED_SHAPE;
  if (!grace_aligned16(logits) || (reinterpret_cast<uintptr_t>(ws) & 255u)) return GRACE_INVALID_ARG;
  if (ws_bytes < grace_beam_topk_workspace_bytes(B, N, K)) return GRACE_WORKSPACE_TOO_SMALL;
  int log2_V = -1;
  if ((V & (V - 1)) == 0)
    for (log2_V = 0; (1 << log2_V) < V; ++log2_V) {}
  grace::CandSrc src = {logits, allow_bits, row_score, row_lse, N, V, log2_V};
  return grace::launch_beam_topk(src, B, K, V, out_score, out_flat, out_parent, out_token, ws, d_status,
                                 (cudaStream_t)stream);
}



// ---------------------------------------------------------------------------------------------
// grace_beam_topk_static: the same selection with the scratch memory owned by the library.
//
// Some callers cannot allocate device memory at the point where they need a top-k: code running
// inside a framework that forbids allocation on its hot path, a plug-in that is handed input and
// output buffers and nothing else, a process whose memory pool is already fully committed.  For
// them the per-request headers and candidate lists live in a fixed array in the library's own
// device image.  The array is sized for kStaticMaxRequests requests (about 2 MB); every GPU that
// loads the library holds it until the process exits.
// ---------------------------------------------------------------------------------------------
namespace grace {
constexpr int kStaticMaxRequests = 32;
constexpr size_t kStaticScratchBytes =
    (size_t)kStaticMaxRequests * (sizeof(TopkHeader) + (size_t)kCap * sizeof(uint2));
static __device__ __align__(256) unsigned char g_topk_static_scratch[kStaticScratchBytes];

// In host code the name of a __device__ array is only a stand-in, not a device address: the address
// has to be asked for, once per device, while that device is current.
static void* g_static_scratch_ptr[kMaxDevices] = {nullptr};
static unsigned long long g_static_scratch_devices = 0;

static grace_status_t static_scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GRACE_CUDA_ERROR;
  DeviceSetup su(&g_static_scratch_devices);                // two host threads: the second waits for the first's look-up
  if (su) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_topk_static_scratch) != cudaSuccess || ptr == nullptr) return GRACE_CUDA_ERROR;
    g_static_scratch_ptr[dev] = ptr;
    su.done();
  }
  *out = g_static_scratch_ptr[dev];
  return GRACE_OK;
}
}  // namespace grace

extern "C" int grace_beam_topk_static_max_requests(void) { return grace::kStaticMaxRequests; }

extern "C" grace_status_t grace_beam_topk_static(const float* cand, int B, int64_t N, int K, int V,
                                                 float* out_score, int32_t* out_flat, int32_t* out_parent,
                                                 int32_t* out_token, int32_t* d_status, void* stream) {
  if (!cand || !out_score) return GRACE_INVALID_ARG;
  if (B <= 0 || N <= 0 || N >= (1ll << 31) || K < 1 || V <= 0) return GRACE_INVALID_ARG;
  if (K > grace::kMaxK || (N & 3)) return GRACE_UNSUPPORTED_SHAPE;
  if (B > grace::kStaticMaxRequests) return GRACE_WORKSPACE_TOO_SMALL;     // beyond the built-in scratch
  if (!grace_aligned16(cand)) return GRACE_INVALID_ARG;
  void* scratch = nullptr;
  grace_status_t st = grace::static_scratch_for_current_device(&scratch);
  if (st != GRACE_OK) return st;
  // The kernels (re)initialise every header word they read, so the previous call's contents do not
  // matter; nothing here has to start at zero.
  grace::CandSrc src = {cand, nullptr, nullptr, nullptr, N, V, -1};
  return grace::launch_beam_topk(src, B, K, V, out_score, out_flat, out_parent, out_token, scratch, d_status,
                                 (cudaStream_t)stream);
}
