// Host-side index builders: dense child-bitmask trie (Section 4.4, Appendix A), per-request
// node-eligibility bitmask and prefix Bloom filter (Section 4.1's TM in per-request form).
// Not on the timed path.
#include <string>
#include <unordered_map>
#include <algorithm>
#include <vector>

#include "common.cuh"

namespace {

bool sids_sorted_distinct(const int32_t* sids, int64_t n, int V, int L) {
  for (int64_t i = 0; i < n; ++i) {
    const int32_t* cur = sids + i * L;
    for (int j = 0; j < L; ++j)
      if (cur[j] < 0 || cur[j] >= V) return false;
    if (i == 0) continue;
    const int32_t* prev = cur - L;
    int j = 0;
    while (j < L && prev[j] == cur[j]) ++j;
    if (j == L || prev[j] > cur[j]) return false;
  }
  return true;
}

bool shape_ok(const int32_t* sids, int64_t n, int V, int L) {
  return sids != nullptr && n > 0 && V > 0 && V % 64 == 0 && V < 65535 && L >= 1 && L <= 4;
}

// For sorted SIDs, SID i opens a new node at level l (1-based) iff it differs from SID i-1
// somewhere in its first l tokens.  first_diff = index of the first differing token.
inline int first_diff(const int32_t* sids, int64_t i, int L) {
  if (i == 0) return 0;
  const int32_t* a = sids + (i - 1) * L;
  const int32_t* b = sids + i * L;
  int j = 0;
  while (j < L && a[j] == b[j]) ++j;
  return j;
}

inline uint64_t prefix_key(const int32_t* tok, int len) {
  uint64_t key = 0;
  for (int i = 0; i < len; ++i) key |= (uint64_t)(tok[i] + 1) << (16 * i);
  return key;
}

}  // namespace

extern "C" grace_status_t grace_trie_count_nodes(const int32_t* sids, int64_t n_sids, int V, int L,
                                                 int64_t* level_start) {
  if (!shape_ok(sids, n_sids, V, L) || level_start == nullptr) return GRACE_INVALID_ARG;
  if (!sids_sorted_distinct(sids, n_sids, V, L)) return GRACE_INVALID_ARG;
  std::vector<int64_t> count(L + 1, 0);
  count[0] = 1;
  for (int64_t i = 0; i < n_sids; ++i) {
    int d = first_diff(sids, i, L);
    for (int l = d + 1; l <= L; ++l) ++count[l];      // new nodes at levels d+1 .. L
  }
  level_start[0] = 0;
  for (int l = 0; l <= L; ++l) level_start[l + 1] = level_start[l] + count[l];
  return GRACE_OK;
}

extern "C" grace_status_t grace_trie_build_dense(const int32_t* sids, int64_t n_sids, int V, int L,
                                                 uint64_t* child_bits, int32_t* child_base) {
  if (child_bits == nullptr || child_base == nullptr) return GRACE_INVALID_ARG;
  std::vector<int64_t> level_start(L + 2);
  grace_status_t st = grace_trie_count_nodes(sids, n_sids, V, L, level_start.data());
  if (st != GRACE_OK) return st;
  const int64_t n_internal = level_start[L];
  const int W = V / 64;
  for (int64_t i = 0; i < n_internal * W; ++i) child_bits[i] = 0;
  for (int64_t i = 0; i < n_internal; ++i) child_base[i] = -1;
  // cur[l] = id of the node holding the current SID's length-l prefix
  std::vector<int64_t> cur(L + 1, 0), next_id(L + 1);
  for (int l = 0; l <= L; ++l) next_id[l] = level_start[l];
  cur[0] = 0;
  for (int64_t i = 0; i < n_sids; ++i) {
    const int32_t* s = sids + i * L;
    int d = first_diff(sids, i, L);
    for (int l = d + 1; l <= L; ++l) {
      cur[l] = next_id[l]++;
      const int64_t parent = cur[l - 1];
      const int tok = s[l - 1];
      child_bits[parent * W + (tok >> 6)] |= 1ull << (tok & 63);
      if (child_base[parent] < 0) child_base[parent] = (int32_t)cur[l];
    }
  }
  return GRACE_OK;
}

extern "C" grace_status_t grace_node_bitmask_build(const int32_t* sids, int64_t n_sids, int V, int L,
                                                   const uint8_t* eligible, uint64_t* node_bits) {
  if (eligible == nullptr || node_bits == nullptr) return GRACE_INVALID_ARG;
  std::vector<int64_t> level_start(L + 2);
  grace_status_t st = grace_trie_count_nodes(sids, n_sids, V, L, level_start.data());
  if (st != GRACE_OK) return st;
  const int64_t words = (level_start[L + 1] + 63) / 64;
  for (int64_t i = 0; i < words; ++i) node_bits[i] = 0;
  std::vector<int64_t> cur(L + 1, 0), next_id(L + 1);
  for (int l = 0; l <= L; ++l) next_id[l] = level_start[l];
  for (int64_t i = 0; i < n_sids; ++i) {
    int d = first_diff(sids, i, L);
    for (int l = d + 1; l <= L; ++l) cur[l] = next_id[l]++;
    if (eligible[i]) {
      for (int l = 0; l <= L; ++l) node_bits[cur[l] >> 6] |= 1ull << (cur[l] & 63);
    }
  }
  return GRACE_OK;
}

extern "C" grace_status_t grace_bloom_build(const int32_t* sids, int64_t n_sids, int V, int L,
                                            const uint8_t* eligible, int log2_bits, int n_hashes,
                                            uint64_t* bloom_words) {
  if (!shape_ok(sids, n_sids, V, L) || eligible == nullptr || bloom_words == nullptr)
    return GRACE_INVALID_ARG;
  if (log2_bits < 6 || log2_bits > 32 || n_hashes < 1 || n_hashes > 16) return GRACE_INVALID_ARG;
  const uint64_t m_mask = (1ull << log2_bits) - 1;
  for (uint64_t i = 0; i < (1ull << log2_bits) / 64; ++i) bloom_words[i] = 0;
  for (int64_t i = 0; i < n_sids; ++i) {
    if (!eligible[i]) continue;
    for (int len = 1; len <= L; ++len) {
      const uint64_t z = grace::mix64(prefix_key(sids + i * L, len));
      const uint32_t h1 = (uint32_t)z, h2 = (uint32_t)(z >> 32) | 1u;
      for (int p = 0; p < n_hashes; ++p) {
        const uint64_t pos = (uint32_t)(h1 + (uint32_t)p * h2) & m_mask;
        bloom_words[pos >> 6] |= 1ull << (pos & 63);
      }
    }
  }
  return GRACE_OK;
}

extern "C" grace_status_t grace_trie_walk(const uint64_t* child_bits, const int32_t* child_base,
                                          int V, int L, int64_t num_internal, const int32_t* tokens,
                                          int len, int32_t* node) {
  if (!child_bits || !child_base || !tokens || !node || len < 0 || len > L || V % 64) return GRACE_INVALID_ARG;
  const int W = V / 64;
  int64_t cur = 0;
  for (int i = 0; i < len; ++i) {
    const int tok = tokens[i];
    if (tok < 0 || tok >= V || cur >= num_internal) { *node = -1; return GRACE_OK; }
    const uint64_t* row = child_bits + cur * W;
    if (!((row[tok >> 6] >> (tok & 63)) & 1)) { *node = -1; return GRACE_OK; }
    int rank = 0;
    for (int w = 0; w < (tok >> 6); ++w) rank += __builtin_popcountll(row[w]);
    rank += __builtin_popcountll(row[tok >> 6] & ((1ull << (tok & 63)) - 1));
    cur = child_base[cur] + rank;
  }
  *node = (int32_t)cur;
  return GRACE_OK;
}

namespace {
// Rows are deduplicated by content; ids are given in order of first appearance.
struct RowTable {
  int W;
  std::unordered_map<std::string, int32_t> ids;
  std::vector<uint64_t> rows;
  explicit RowTable(int w) : W(w) {}
  int32_t add(const uint64_t* row) {
    std::string key(reinterpret_cast<const char*>(row), sizeof(uint64_t) * W);
    auto it = ids.find(key);
    if (it != ids.end()) return it->second;
    const int32_t id = (int32_t)ids.size();
    ids.emplace(std::move(key), id);
    rows.insert(rows.end(), row, row + W);
    return id;
  }
};
}  // namespace

extern "C" grace_status_t grace_gtm_index_build(const int32_t* sids, int64_t n_sids, int V, int L,
                                                const int64_t* ad_sid, int64_t n_ads, const uint64_t* ad_bitmask,
                                                int W_bm, const uint64_t* ad_bloom, int W_bl,
                                                int32_t* node_offsets, int32_t* csr_child_nodes, int16_t* csr_tokens,
                                                int32_t* bitmask_index, int32_t* bloom_index,
                                                uint64_t* bitmask_table, int64_t* n_bitmask_rows,
                                                uint64_t* bloom_table, int64_t* n_bloom_rows) {
  if (!ad_sid || !ad_bitmask || !ad_bloom || !node_offsets || !csr_child_nodes || !csr_tokens || !bitmask_index ||
      !bloom_index || !n_bitmask_rows || !n_bloom_rows || n_ads <= 0 || W_bm <= 0 || W_bl <= 0 || V > 32767)
    return GRACE_INVALID_ARG;
  if ((bitmask_table == nullptr) != (bloom_table == nullptr)) return GRACE_INVALID_ARG;
  std::vector<int64_t> level_start(L + 2);
  grace_status_t st = grace_trie_count_nodes(sids, n_sids, V, L, level_start.data());
  if (st != GRACE_OK) return st;
  const int64_t num_nodes = level_start[L + 1];
  // ads: sorted by SID, every SID covered
  for (int64_t a = 0; a < n_ads; ++a) {
    if (ad_sid[a] < 0 || ad_sid[a] >= n_sids || (a > 0 && ad_sid[a] < ad_sid[a - 1])) return GRACE_INVALID_ARG;
    if (a > 0 && ad_sid[a] > ad_sid[a - 1] + 1) return GRACE_INVALID_ARG;
  }
  if (ad_sid[0] != 0 || ad_sid[n_ads - 1] != n_sids - 1) return GRACE_INVALID_ARG;
  // node rows: every node on the path of a SID receives the OR of that SID's ads
  std::vector<uint64_t> node_bm((size_t)num_nodes * W_bm, 0), node_bl((size_t)num_nodes * W_bl, 0);
  std::vector<int64_t> cur(L + 1, 0), next_id(L + 1), parent_of((size_t)num_nodes, -1);
  std::vector<int16_t> token_of((size_t)num_nodes, 0);
  for (int l = 0; l <= L; ++l) next_id[l] = level_start[l];
  int64_t a = 0;
  for (int64_t i = 0; i < n_sids; ++i) {
    const int d = first_diff(sids, i, L);
    for (int l = d + 1; l <= L; ++l) {
      cur[l] = next_id[l]++;
      parent_of[cur[l]] = cur[l - 1];
      token_of[cur[l]] = (int16_t)sids[i * L + l - 1];
    }
    for (; a < n_ads && ad_sid[a] == i; ++a) {
      for (int l = 0; l <= L; ++l) {
        uint64_t* bm = &node_bm[(size_t)cur[l] * W_bm];
        uint64_t* bl = &node_bl[(size_t)cur[l] * W_bl];
        for (int w = 0; w < W_bm; ++w) bm[w] |= ad_bitmask[a * W_bm + w];
        for (int w = 0; w < W_bl; ++w) bl[w] |= ad_bloom[a * W_bl + w];
      }
    }
  }
  // child entries in node order: entry j leads to node j + 1 (level order, lexicographic inside a level)
  for (int64_t n = 0; n <= num_nodes; ++n) node_offsets[n] = 0;
  for (int64_t c = 1; c < num_nodes; ++c) ++node_offsets[parent_of[c] + 1];
  for (int64_t n = 0; n < num_nodes; ++n) node_offsets[n + 1] += node_offsets[n];
  RowTable bm_rows(W_bm), bl_rows(W_bl);
  for (int64_t c = 1; c < num_nodes; ++c) {
    const int64_t j = c - 1;
    csr_child_nodes[j] = (int32_t)c;
    csr_tokens[j] = token_of[c];
    bitmask_index[j] = bm_rows.add(&node_bm[(size_t)c * W_bm]);
    bloom_index[j] = bl_rows.add(&node_bl[(size_t)c * W_bl]);
  }
  if (bitmask_table != nullptr) {
    if (*n_bitmask_rows < (int64_t)bm_rows.ids.size() || *n_bloom_rows < (int64_t)bl_rows.ids.size())
      return GRACE_WORKSPACE_TOO_SMALL;
    std::copy(bm_rows.rows.begin(), bm_rows.rows.end(), bitmask_table);
    std::copy(bl_rows.rows.begin(), bl_rows.rows.end(), bloom_table);
  }
  *n_bitmask_rows = (int64_t)bm_rows.ids.size();
  *n_bloom_rows = (int64_t)bl_rows.ids.size();
  return GRACE_OK;
}

namespace {
inline int popcount_row(const uint64_t* a, const uint64_t* b, int W) {   // set bits of a | b
  int n = 0;
  for (int w = 0; w < W; ++w) n += __builtin_popcountll(a[w] | b[w]);
  return n;
}
// Greedy split of the SIDs [lo, hi) into at most k groups (smallest fill after the OR, lowest group on
// ties).  Group rows are written to g_bm / g_bl ([k][W]); returns the largest group popcount and marks
// the groups that received a SID.
int greedy_groups(const uint64_t* leaf_bm, const uint64_t* leaf_bl, int64_t lo, int64_t hi, int k, int W_bm, int W_bl,
                  std::vector<uint64_t>& g_bm, std::vector<uint64_t>& g_bl, std::vector<char>& used) {
  g_bm.assign((size_t)k * W_bm, 0);
  g_bl.assign((size_t)k * W_bl, 0);
  used.assign(k, 0);
  for (int64_t i = lo; i < hi; ++i) {
    int best = 0, best_pc = 1 << 30;
    for (int g = 0; g < k; ++g) {
      const int pc = popcount_row(&g_bm[(size_t)g * W_bm], leaf_bm + i * W_bm, W_bm) +
                     popcount_row(&g_bl[(size_t)g * W_bl], leaf_bl + i * W_bl, W_bl);
      if (pc < best_pc) { best_pc = pc; best = g; }
    }
    for (int w = 0; w < W_bm; ++w) g_bm[(size_t)best * W_bm + w] |= leaf_bm[i * W_bm + w];
    for (int w = 0; w < W_bl; ++w) g_bl[(size_t)best * W_bl + w] |= leaf_bl[i * W_bl + w];
    used[best] = 1;
  }
  int max_pc = 0;
  for (int g = 0; g < k; ++g) {
    if (!used[g]) continue;
    int pc = 0;
    for (int w = 0; w < W_bm; ++w) pc += __builtin_popcountll(g_bm[(size_t)g * W_bm + w]);
    for (int w = 0; w < W_bl; ++w) pc += __builtin_popcountll(g_bl[(size_t)g * W_bl + w]);
    if (pc > max_pc) max_pc = pc;
  }
  return max_pc;
}
}  // namespace

extern "C" grace_status_t grace_gtm_index_build_kway(const int32_t* sids, int64_t n_sids, int V, int L,
                                                     const int64_t* ad_sid, int64_t n_ads, const uint64_t* ad_bitmask,
                                                     int W_bm, const uint64_t* ad_bloom, int W_bl,
                                                     const int32_t* k_level, double fill_target, int k_max,
                                                     int32_t* node_offsets, int32_t* csr_child_nodes,
                                                     int16_t* csr_tokens, int32_t* part_offsets,
                                                     int32_t* part_bitmask_index, int32_t* part_bloom_index,
                                                     int64_t* n_parts, uint64_t* bitmask_table, int64_t* n_bitmask_rows,
                                                     uint64_t* bloom_table, int64_t* n_bloom_rows) {
  if (!ad_sid || !ad_bitmask || !ad_bloom || !node_offsets || !csr_child_nodes || !csr_tokens || !part_offsets ||
      !n_parts || !n_bitmask_rows || !n_bloom_rows || n_ads <= 0 || W_bm <= 0 || W_bl <= 0 || V > 32767)
    return GRACE_INVALID_ARG;
  const bool sizing = (part_bitmask_index == nullptr);
  if ((part_bloom_index == nullptr) != sizing || (bitmask_table == nullptr) != sizing || (bloom_table == nullptr) != sizing)
    return GRACE_INVALID_ARG;
  if (k_level == nullptr && k_max < 1) return GRACE_INVALID_ARG;
  if (k_level != nullptr)
    for (int l = 1; l <= L; ++l)
      if (k_level[l] < 1) return GRACE_INVALID_ARG;
  std::vector<int64_t> level_start(L + 2);
  grace_status_t st = grace_trie_count_nodes(sids, n_sids, V, L, level_start.data());
  if (st != GRACE_OK) return st;
  const int64_t num_nodes = level_start[L + 1];
  for (int64_t a = 0; a < n_ads; ++a) {
    if (ad_sid[a] < 0 || ad_sid[a] >= n_sids || (a > 0 && ad_sid[a] < ad_sid[a - 1])) return GRACE_INVALID_ARG;
    if (a > 0 && ad_sid[a] > ad_sid[a - 1] + 1) return GRACE_INVALID_ARG;
  }
  if (ad_sid[0] != 0 || ad_sid[n_ads - 1] != n_sids - 1) return GRACE_INVALID_ARG;
  // rows of a SID: OR over its ads
  std::vector<uint64_t> leaf_bm((size_t)n_sids * W_bm, 0), leaf_bl((size_t)n_sids * W_bl, 0);
  for (int64_t a = 0; a < n_ads; ++a) {
    for (int w = 0; w < W_bm; ++w) leaf_bm[(size_t)ad_sid[a] * W_bm + w] |= ad_bitmask[a * W_bm + w];
    for (int w = 0; w < W_bl; ++w) leaf_bl[(size_t)ad_sid[a] * W_bl + w] |= ad_bloom[a * W_bl + w];
  }
  // trie structure (as in grace_gtm_index_build) and, per node, the run of SIDs below it
  std::vector<int64_t> cur(L + 1, 0), next_id(L + 1), parent_of((size_t)num_nodes, -1);
  std::vector<int64_t> sid_lo((size_t)num_nodes, 0), sid_hi((size_t)num_nodes, 0);
  std::vector<int16_t> token_of((size_t)num_nodes, 0);
  std::vector<int8_t> level_of((size_t)num_nodes, 0);
  for (int l = 0; l <= L; ++l) next_id[l] = level_start[l];
  for (int64_t i = 0; i < n_sids; ++i) {
    const int d = first_diff(sids, i, L);
    for (int l = d + 1; l <= L; ++l) {
      cur[l] = next_id[l]++;
      parent_of[cur[l]] = cur[l - 1];
      token_of[cur[l]] = (int16_t)sids[i * L + l - 1];
      level_of[cur[l]] = (int8_t)l;
      sid_lo[cur[l]] = i;
    }
    for (int l = 1; l <= L; ++l) sid_hi[cur[l]] = i + 1;
  }
  for (int64_t n = 0; n <= num_nodes; ++n) node_offsets[n] = 0;
  for (int64_t c = 1; c < num_nodes; ++c) ++node_offsets[parent_of[c] + 1];
  for (int64_t n = 0; n < num_nodes; ++n) node_offsets[n + 1] += node_offsets[n];
  RowTable bm_rows(W_bm), bl_rows(W_bl);
  std::vector<uint64_t> g_bm, g_bl;
  std::vector<char> used;
  const int bits = 64 * (W_bm + W_bl);
  int64_t slot = 0;
  part_offsets[0] = 0;
  for (int64_t c = 1; c < num_nodes; ++c) {
    const int64_t j = c - 1, lo = sid_lo[c], hi = sid_hi[c];
    csr_child_nodes[j] = (int32_t)c;
    csr_tokens[j] = token_of[c];
    int k;
    if (k_level != nullptr) {
      k = (int)std::max<int64_t>(1, std::min<int64_t>(k_level[level_of[c]], hi - lo));
      greedy_groups(leaf_bm.data(), leaf_bl.data(), lo, hi, k, W_bm, W_bl, g_bm, g_bl, used);
    } else {
      const int k_top = (int)std::max<int64_t>(1, std::min<int64_t>(k_max, hi - lo));
      for (k = 1; k <= k_top; ++k) {
        const int max_pc = greedy_groups(leaf_bm.data(), leaf_bl.data(), lo, hi, k, W_bm, W_bl, g_bm, g_bl, used);
        if ((double)max_pc / (double)bits <= fill_target || k == k_top) break;
      }
    }
    for (int g = 0; g < k; ++g) {
      if (!used[g]) continue;
      const int32_t ib = bm_rows.add(&g_bm[(size_t)g * W_bm]), il = bl_rows.add(&g_bl[(size_t)g * W_bl]);
      if (!sizing) {
        if (slot >= *n_parts) return GRACE_WORKSPACE_TOO_SMALL;
        part_bitmask_index[slot] = ib;
        part_bloom_index[slot] = il;
      }
      ++slot;
    }
    if (slot > 0x7fffffff) return GRACE_UNSUPPORTED_SHAPE;
    part_offsets[j + 1] = (int32_t)slot;
  }
  if (!sizing) {
    if (*n_bitmask_rows < (int64_t)bm_rows.ids.size() || *n_bloom_rows < (int64_t)bl_rows.ids.size())
      return GRACE_WORKSPACE_TOO_SMALL;
    std::copy(bm_rows.rows.begin(), bm_rows.rows.end(), bitmask_table);
    std::copy(bl_rows.rows.begin(), bl_rows.rows.end(), bloom_table);
  }
  *n_parts = slot;
  *n_bitmask_rows = (int64_t)bm_rows.ids.size();
  *n_bloom_rows = (int64_t)bl_rows.ids.size();
  return GRACE_OK;
}

extern "C" const char* grace_status_string(grace_status_t s) {
  switch (s) {
    case GRACE_OK: return "ok";
    case GRACE_INVALID_ARG: return "invalid argument";
    case GRACE_UNSUPPORTED_SHAPE: return "unsupported shape";
    case GRACE_WORKSPACE_TOO_SMALL: return "workspace too small";
    case GRACE_CUDA_ERROR: return "CUDA error";
    case GRACE_TIMEOUT: return "timeout";
  }
  return "unknown";
}

unsigned long long g_grace_launches = 0;
extern "C" uint64_t grace_kernel_launch_count(void) { return __atomic_load_n(&g_grace_launches, __ATOMIC_RELAXED); }
extern "C" int grace_version(void) { return 1; }
extern "C" int grace_built_for_sm(void) { return 100; }

// ------------------------------------------------------------------------------------------------
// Weight preparation for the folded-LayerNorm decode path (host memory in, host memory out)
// ------------------------------------------------------------------------------------------------
namespace {
inline uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);   // NaN stays NaN
  u += 0x7fffu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}
inline float bf16_to_f32(uint16_t b) {
  const uint32_t u = (uint32_t)b << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}
}  // namespace

extern "C" grace_status_t grace_f32_to_bf16(const float* a, int64_t n, uint16_t* out) {
  if (!a || !out || n < 0) return GRACE_INVALID_ARG;
  for (int64_t i = 0; i < n; ++i) out[i] = f32_to_bf16_rne(a[i]);
  return GRACE_OK;
}

extern "C" grace_status_t grace_fold_layer_norm(const float* w, const float* gamma, const float* beta,
                                                int64_t N, int64_t K, uint16_t* w_folded, float* col_sum,
                                                float* col_bias) {
  if (!w || !gamma || !beta || !w_folded || !col_sum || !col_bias || N <= 0 || K <= 0) return GRACE_INVALID_ARG;
  for (int64_t n = 0; n < N; ++n) {
    double cs = 0.0, cb = 0.0;
    for (int64_t k = 0; k < K; ++k) {
      const float wv = w[n * K + k];
      const uint16_t b = f32_to_bf16_rne(wv * gamma[k]);       // the operand the GEMM will multiply with
      w_folded[n * K + k] = b;
      cs += (double)bf16_to_f32(b);                              // column sums of exactly those operands
      cb += (double)wv * (double)beta[k];
    }
    col_sum[n] = (float)cs;
    col_bias[n] = (float)cb;
  }
  return GRACE_OK;
}

extern "C" grace_status_t grace_centre_rows(const float* a, int64_t n, int64_t d, float* out) {
  if (!a || !out || n <= 0 || d <= 0) return GRACE_INVALID_ARG;
  for (int64_t i = 0; i < n; ++i) {
    double m = 0.0;
    for (int64_t j = 0; j < d; ++j) m += (double)a[i * d + j];
    m /= (double)d;
    for (int64_t j = 0; j < d; ++j) out[i * d + j] = (float)((double)a[i * d + j] - m);
  }
  return GRACE_OK;
}

extern "C" grace_status_t grace_centre_outputs(const float* w, int64_t d_out, int64_t K, float* out) {
  if (!w || !out || d_out <= 0 || K <= 0) return GRACE_INVALID_ARG;
  std::vector<double> m((size_t)K, 0.0);
  for (int64_t i = 0; i < d_out; ++i)
    for (int64_t k = 0; k < K; ++k) m[(size_t)k] += (double)w[i * K + k];
  for (int64_t k = 0; k < K; ++k) m[(size_t)k] /= (double)d_out;
  for (int64_t i = 0; i < d_out; ++i)
    for (int64_t k = 0; k < K; ++k) out[i * K + k] = (float)((double)w[i * K + k] - m[(size_t)k]);
  return GRACE_OK;
}
