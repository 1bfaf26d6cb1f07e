/*
 * grace.h -- C ABI of the B200 decode-step library (libgrace_b200.so).
 *
 * One decode step of a GTM-constrained, wide-beam, short-sequence SID decoder
 * (GRACE, Sections 3.1-3.3, 4.1-4.4, 5.1-5.4):
 *
 *   cross-attention  beams of a request as query rows against shared K/V   grace_cross_attn
 *   self-attention   over a parent-addressed KV cache, fused cache write   grace_self_attn
 *   CD + GTM mask    and score add on next-token log-probabilities          grace_gtm_mask
 *   beam top-k       per request over beam x codebook candidates            grace_beam_topk
 *   state update     node ids / keys of the selected children               grace_beam_update
 *   whole step       decoder layers + the four ops above                    grace_decode_step
 *
 * Conventions (all functions):
 *   - Pointers named d_* or documented "device" are device pointers; "host" are host pointers.
 *   - Every buffer is caller-owned; the library never allocates or frees device memory and
 *     never synchronises.  Work is enqueued on `stream` (a cudaStream_t passed as void*); the
 *     buffers must stay alive until the stream has passed the call.
 *   - Rows are request-major: row r = b * M + m (Appendix B).
 *   - Return value: GRACE_OK or an error detected on the host before anything is enqueued.
 *   - `d_status` (device int32*, may be NULL): conditions detected on the device are OR-ed
 *     into it (GRACE_DEV_* bits).  The caller zeroes it.
 *   - bf16 tensors are passed as uint16_t* holding bf16 bit patterns.
 */
#ifndef GRACE_H_
#define GRACE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  GRACE_OK = 0,
  GRACE_INVALID_ARG = 1,        /* null pointer, misaligned pointer, negative size         */
  GRACE_UNSUPPORTED_SHAPE = 2,  /* shape outside what the kernels are built for            */
  GRACE_WORKSPACE_TOO_SMALL = 3,
  GRACE_CUDA_ERROR = 4,         /* a CUDA runtime / driver call failed                     */
  GRACE_TIMEOUT = 5
} grace_status_t;

/* bits OR-ed into *d_status by kernels */
#define GRACE_DEV_BAD_INDEX 1   /* a gathered index was out of range; the access was skipped */
#define GRACE_DEV_NAN 2         /* NaN among log-probs / candidates (precondition violated)   */
#define GRACE_DEV_TIMEOUT 4     /* a bounded device-side wait ran out                        */
#define GRACE_DEV_TOPK_EXACT_PATH 8 /* informational: top-k fell back to the multi-pass path  */

const char* grace_status_string(grace_status_t s);
/* Library version, and the compute capability the kernels were built for (100 = sm_100a). */
int grace_version(void);
int grace_built_for_sm(void);
/* Every device-side wait of the tensor-core kernels (on an mbarrier that TMA, the tensor cores or a peer
 * CTA completes) is bounded: after about a second it gives up, the kernel's remaining waits return at
 * once, the kernel frees its TMEM and exits, and the output of that launch is undefined.
 * grace_wait_timeouts: number of waits that gave up on the current device since the previous call
 * (0 in normal operation; -1 if the counter cannot be read).  Synchronize the streams first.
 * grace_selftest_bounded_wait: runs a one-block kernel that waits (limit: about a millisecond) on a
 * barrier nothing arrives on, synchronizes `stream`, and returns GRACE_TIMEOUT when the wait gave up as
 * designed (grace_wait_timeouts then reports it); the context stays usable. */
int grace_wait_timeouts(void);
grace_status_t grace_selftest_bounded_wait(void* stream);

/* Asks the device to keep `fraction` (0 < fraction <= 1) of the lines of [ptr, ptr + bytes) resident in L2 for
 * the kernels launched on `stream` from now on: an access-policy window on the stream (hit ratio = fraction,
 * other lines of the window cached normally), backed by this context's persisting-L2 carve-out, both clipped
 * to the device's limits.  Meant for the residual stream of the decoder, which every block of a step re-reads
 * several times while far larger tensors stream past it; keeping all of a buffer half the size of the L2
 * starves everything else (measured: slower), half of it pays.  ptr NULL or bytes 0 clears the window.
 * Host call; nothing is enqueued; the setting belongs to this process's context and ends with it.
 * GRACE_UNSUPPORTED_SHAPE if the device has no persisting L2. */
grace_status_t grace_stream_l2_persist(void* stream, const void* ptr, size_t bytes, float fraction);

/* Number of kernels this library has launched in this process so far (all entry points). */
uint64_t grace_kernel_launch_count(void);

/* ------------------------------------------------------------------------------------------
 * Index structures (Section 4.4, Appendix A).
 *
 * The trie is held in its per-node child-bitmask form: node ids are assigned level by level
 * (root = 0) and, inside a level, in lexicographic prefix order, so the children of a node are
 * consecutive ids in token order and
 *     child(n, v) = child_base[n] + popcount(child_bits[n] restricted to tokens < v).
 * CD_t[v] (Section 4.1) is bit v of child_bits[n].  Only nodes of levels 0..L-1 have rows.
 * ---------------------------------------------------------------------------------------- */
typedef struct {
  int32_t V;                    /* vocabulary size per position; multiple of 64, <= 65535 - 1 */
  int32_t L;                    /* SID length                                             */
  int64_t num_nodes;            /* all nodes, leaves included                             */
  int64_t num_internal;         /* nodes of levels 0..L-1 (those with rows below)         */
  const uint64_t* child_bits;   /* device [num_internal][V/64]; token v = bit v&63 of word v>>6 */
  const int32_t* child_base;    /* device [num_internal]; id of the first child, -1 if none */
} grace_trie_t;

typedef enum {
  GRACE_MATCH_NONE = 0,         /* TM = 1: constrained decoding only                      */
  GRACE_MATCH_NODE_BITMASK = 1, /* per request, one eligibility bit per trie node         */
  GRACE_MATCH_PREFIX_BLOOM = 2  /* per request, a Bloom filter over prefix keys           */
} grace_matcher_kind_t;

/* TM_t[v] = match(u, p || v) (Section 4.1) in its per-request forms.
 *   NODE_BITMASK: bits = device uint64 [B][words_per_request]; node n is bit n&63 of word n>>6;
 *                 a prefix is eligible iff its subtree holds an eligible SID.
 *   PREFIX_BLOOM: bits = device uint64 [B][words_per_request], words_per_request = 2^log2_bits/64.
 *                 key(p) = sum_i (token_i + 1) << 16 i;  z = splitmix64 finaliser of key;
 *                 h1 = low 32 bits, h2 = high 32 bits | 1; probe_i = (h1 + i*h2) mod 2^32 mod 2^log2_bits,
 *                 i = 0 .. n_hashes-1.  Member iff all probed bits are set. */
typedef struct {
  int32_t kind;
  int32_t bloom_log2_bits;
  int32_t bloom_hashes;
  int32_t reserved;
  int64_t words_per_request;
  const uint64_t* bits;
} grace_matcher_t;

/* Host-side index builders (not on the timed path; host memory in, host memory out).
 * `sids` is host int32 [n_sids][L], lexicographically sorted and distinct (else INVALID_ARG). */

/* level_start: host int64 [L+2]; level_start[l] = id of the first node of level l,
 * level_start[L+1] = num_nodes. */
grace_status_t grace_trie_count_nodes(const int32_t* sids, int64_t n_sids, int V, int L,
                                      int64_t* level_start);
/* child_bits host uint64 [level_start[L]][V/64], child_base host int32 [level_start[L]]. */
grace_status_t grace_trie_build_dense(const int32_t* sids, int64_t n_sids, int V, int L,
                                      uint64_t* child_bits, int32_t* child_base);
/* node_bits host uint64 [ceil(num_nodes/64)], zeroed by the callee: upward closure of the
 * eligible SIDs (eligible: host uint8 [n_sids], non-zero = eligible). */
grace_status_t grace_node_bitmask_build(const int32_t* sids, int64_t n_sids, int V, int L,
                                        const uint8_t* eligible, uint64_t* node_bits);
/* bloom_words host uint64 [2^log2_bits / 64], zeroed by the callee: keys of every prefix
 * (length 1..L) of every eligible SID. */
grace_status_t grace_bloom_build(const int32_t* sids, int64_t n_sids, int V, int L,
                                 const uint8_t* eligible, int log2_bits, int n_hashes,
                                 uint64_t* bloom_words);
/* Node id of a prefix (host tokens[len]) in a host copy of the dense trie; *node = -1 if the
 * prefix is not in the catalog. */
grace_status_t grace_trie_walk(const uint64_t* child_bits, const int32_t* child_base, int V, int L,
                               int64_t num_internal, const int32_t* tokens, int len, int32_t* node);

/* ------------------------------------------------------------------------------------------
 * Weight preparation for the folded-LayerNorm decode path (host memory in, host memory out; not
 * on the timed path).  No passage of the paper defines these: Section 3.2 fixes neither the
 * normalisation nor its placement; the decoder here is pre-LayerNorm, and two identities of a
 * pre-LayerNorm block are used to take the LayerNorm kernels off the path:
 *   (fold)    LN(x; gamma, beta) W^T = rstd (x W'^T) - rstd mean colsum(W') + W beta,
 *             W' = W * gamma (column-wise), rstd = 1 / sqrt(var(x) + eps)  (per row of x);
 *   (centre)  LayerNorm does not see a per-row shift of its input, so everything ADDED into the
 *             residual stream may be centred over the feature axis; the stream's rows then keep
 *             zero mean and the colsum term vanishes.
 * grace_decode_step with row_affine set expects weights prepared by these helpers.
 *
 * grace_fold_layer_norm:  w host fp32 [N, K] (row n = output feature n), gamma, beta host fp32 [K].
 *   w_folded  host bf16 [N, K] = round-to-nearest-even(w[n,k] * gamma[k])   (the GEMM's operand)
 *   col_sum   host fp32 [N]    = sum_k of the ROUNDED w_folded[n,k]           (fp64 accumulation)
 *   col_bias  host fp32 [N]    = sum_k w[n,k] * beta[k]                       (fp64 accumulation)
 * grace_centre_rows:     a host fp32 [n, d] -> out[i, :] = a[i, :] - mean(a[i, :])   (embedding, position rows)
 * grace_centre_outputs:  w host fp32 [d_out, K] (a projection INTO the stream: row i = stream
 *   feature i) -> out[i, k] = w[i, k] - mean_i(w[i, k]): every output row of x W^T then has zero mean.
 * grace_f32_to_bf16:     round-to-nearest-even conversion, host fp32 [n] -> host bf16 [n].
 * out may alias the input in the two centring calls.  Errors: GRACE_INVALID_ARG for null pointers
 * or non-positive sizes; nothing else can fail.
 * ---------------------------------------------------------------------------------------- */
grace_status_t grace_fold_layer_norm(const float* w, const float* gamma, const float* beta, int64_t N, int64_t K,
                                     uint16_t* w_folded, float* col_sum, float* col_bias);
grace_status_t grace_centre_rows(const float* a, int64_t n, int64_t d, float* out);
grace_status_t grace_centre_outputs(const float* w, int64_t d_out, int64_t K, float* out);
grace_status_t grace_f32_to_bf16(const float* a, int64_t n, uint16_t* out);

/* ------------------------------------------------------------------------------------------
 * Cross-attention, beam-as-query layout (Section 5.1, Appendix B).
 *   out[b*M+m, h, :] = softmax_t( q[b*M+m, h, :] . k[b, h, t, :] * scale ) @ v[b, h, :, :]
 * K and V are read once per (request, head) and shared by the M beams of the request.
 *   q, out : device bf16, element (r, h, i) at r*row_stride + h*d_h + i   (strides in elements)
 *   k, v   : device bf16, element (b, h, t, i) at b*kv_stride_b + h*kv_stride_h + t*kv_stride_t + i
 *   lse    : device fp32 [B*M][H] or NULL; natural-log sum-exp of the scaled scores
 * fp32 accumulation and softmax; bf16 output.  Pointers 16-byte aligned, strides multiples of 8.
 * Supported: d_h in {32, 64, 128}; any B, M, H, T_ctx >= 1.
 * ---------------------------------------------------------------------------------------- */
grace_status_t grace_cross_attn(const uint16_t* q, int64_t q_row_stride,
                                const uint16_t* k, const uint16_t* v,
                                int64_t kv_stride_b, int64_t kv_stride_h, int64_t kv_stride_t,
                                uint16_t* out, int64_t out_row_stride, float* lse,
                                int B, int M, int H, int d_h, int T_ctx, float scale,
                                int32_t* d_status, void* stream);

/* The same with padded encoder outputs (an extension; the paper fixes T_ctx per batch, Section 3.2):
 *   enc_len : device int32 [B] or NULL; request b attends to positions 0 .. enc_len[b]-1 only
 *             (values are clamped to [0, T_ctx]); NULL = all T_ctx positions.
 * A request with enc_len 0 gets zero output rows and lse = -inf (the softmax over an empty set is
 * left undefined by the paper).  grace_cross_attn is this call with enc_len = NULL. */
grace_status_t grace_cross_attn_varlen(const uint16_t* q, int64_t q_row_stride,
                                       const uint16_t* k, const uint16_t* v,
                                       int64_t kv_stride_b, int64_t kv_stride_h, int64_t kv_stride_t,
                                       uint16_t* out, int64_t out_row_stride, float* lse,
                                       const int32_t* enc_len,
                                       int B, int M, int H, int d_h, int T_ctx, float scale,
                                       int32_t* d_status, void* stream);

/* ------------------------------------------------------------------------------------------
 * Self-attention over the parent-addressed KV cache, fused with the cache write
 * (Sections 5.2, 5.3; the block table P of Section 5.3 in its uncomposed form).
 * Row r = b*M_t + m at step t:
 *   k_cache[t][r] <- k of qkv[r],  v_cache[t][r] <- v of qkv[r]
 *   a_t = m;  a_{j-1} = parents[j][b*M_j + a_j]          (j = t .. 1)
 *   out[r, h] = softmax_j( q[r,h] . k_cache[j][b*M_j + a_j, h] * scale ) @ v_cache[j][...],  j = 0..t
 * The current token is part of the prefix; no KV bytes are ever copied on beam reordering.
 *   qkv     : device bf16 [R][3][H][d_h], row stride qkv_row_stride elements
 *   k_cache, v_cache : device bf16 [L_cache][R_max][H][d_h]
 *   parents : device int32 [L_cache][R_max]; slab j (j >= 1) holds, for each row of step j, the
 *             index of its parent inside the same request's step-(j-1) beam; slab 0 is unused
 *   beam_sizes : host int32 [t+1] = M_0 .. M_t
 *   out     : device bf16 [R][H][d_h], row stride out_row_stride elements
 * Supported: t <= 7, d_h in {32, 64, 128}, H*d_h a multiple of 8 and <= 2048.
 * An out-of-range parent index sets GRACE_DEV_BAD_INDEX and is treated as 0.
 * ---------------------------------------------------------------------------------------- */
grace_status_t grace_self_attn(const uint16_t* qkv, int64_t qkv_row_stride,
                               uint16_t* k_cache, uint16_t* v_cache,
                               const int32_t* parents, const int32_t* beam_sizes,
                               uint16_t* out, int64_t out_row_stride,
                               int B, int t, int H, int d_h, int64_t R_max, float scale,
                               int32_t* d_status, void* stream);
/* The same with the cache held in place: qkv_slabs is device bf16 [L_cache][R_max][3][H][d_h] (row stride
 * row_stride >= 3*H*d_h elements, slab stride slab_stride >= R_max*row_stride elements), slab j being the QKV
 * projection of step j exactly as the GEMM left it.  Slab t is this step's input; the K and V thirds of slabs
 * 0..t are the cache, so nothing is copied and the kernel writes only `out` (Section 5.3 removes the reorder
 * copy; this also removes the append copy).  Other arguments, limits and errors as grace_self_attn. */
grace_status_t grace_self_attn_inplace(uint16_t* qkv_slabs, int64_t row_stride, int64_t slab_stride,
                                       const int32_t* parents, const int32_t* beam_sizes,
                                       uint16_t* out, int64_t out_row_stride,
                                       int B, int t, int H, int d_h, int64_t R_max, float scale,
                                       int32_t* d_status, void* stream);

/* ------------------------------------------------------------------------------------------
 * CD + GTM mask and score add (Sections 3.1, 4.1; kernel role of Section 5.4).
 *   allow[r, v] = CD(node[r], v) AND TM(b, prefix[r] || v)
 *   cand[r, v]  = beam_score[r] + logp[r, v] (one fp32 add) if allow else -inf
 *   logp fp32 [R][V]; beam_score fp32 [R]; beam_node int32 [R] (-1 = dead beam: nothing allowed);
 *   beam_key uint64 [R] (prefix keys, read only by the Bloom matcher); prefix_len = tokens
 *   already decoded (= step index).  cand fp32 [R][V] (may be NULL), allow_bits uint64 [R][V/64]
 *   (may be NULL).  All device.  R = B*M.
 * ---------------------------------------------------------------------------------------- */
grace_status_t grace_gtm_mask(const float* logp, const float* beam_score, const int32_t* beam_node,
                              const uint64_t* beam_key, const grace_trie_t* trie,
                              const grace_matcher_t* matcher, float* cand, uint64_t* allow_bits,
                              int B, int M, int V, int prefix_len, int32_t* d_status, void* stream);

/* The same with the log-softmax fused in (Section 3.1: "a fused constraint kernel"): `logits` fp32
 * [R][V] are raw decoder outputs; each live row is read once, normalised over the whole vocabulary
 * (log-sum-exp written to row_lse fp32 [R] if not NULL, 0 for dead rows) and
 *   cand[r, v] = beam_score[r] + (logits[r, v] - lse[r]) if allowed else -inf.
 * cand may alias logits. */
grace_status_t grace_gtm_mask_logits(const float* logits, float* row_lse, const float* beam_score,
                                     const int32_t* beam_node, const uint64_t* beam_key,
                                     const grace_trie_t* trie, const grace_matcher_t* matcher,
                                     float* cand, uint64_t* allow_bits, int B, int M, int V,
                                     int prefix_len, int32_t* d_status, void* stream);

/* grace_gtm_mask_logits with the rows' sums already started by the producer of the logits: lse_part fp32
 * [B*M][n_parts][2] holds, per row and column tile, (maximum, sum of e^(x - maximum)) as written by
 * grace_linear_f32_lse (n_parts = V / 256 <= 32).  The kernel merges them instead of reading the row, so with
 * cand = NULL it does not touch the logits at all. */
grace_status_t grace_gtm_mask_logits_parts(const float* logits, float* row_lse, const float* beam_score,
                                           const int32_t* beam_node, const uint64_t* beam_key,
                                           const grace_trie_t* trie, const grace_matcher_t* matcher,
                                           float* cand, uint64_t* allow_bits, int B, int M, int V,
                                           int prefix_len, const float* lse_part, int n_parts,
                                           int32_t* d_status, void* stream);

/* The constraint alone (Sections 3.1, 4.1): allow_bits[r][V / 64] = catalog-valid children of the row's node AND
 * the request's matcher, exactly the bits grace_gtm_mask* leave, computed from the beam state only.  It needs
 * no log-probabilities, so it can run BEFORE the logits GEMM of a decode step, which then stores only the
 * allowed logits (grace_linear_logits_allowed): the [B*M][V] fp32 tensor is never written out.
 * Arguments and errors as grace_gtm_mask. */
grace_status_t grace_gtm_allow_bits(const int32_t* beam_node, const uint64_t* beam_key, const grace_trie_t* trie,
                                    const grace_matcher_t* matcher, uint64_t* allow_bits, int B, int M, int V,
                                    int prefix_len, int32_t* d_status, void* stream);

/* row_lse[r] = log-sum-exp of row r from the per-tile partials lse_part [R][n_parts][2] of a logits GEMM
 * (n_parts <= 32), 0 for dead rows (beam_node < 0 or a leaf): the merge grace_gtm_mask_logits_parts performs,
 * bit for bit, as a kernel of its own for the order allow bits -> GEMM -> merge -> selection. */
grace_status_t grace_row_lse_from_parts(const float* lse_part, int n_parts, const int32_t* beam_node,
                                        const grace_trie_t* trie, float* row_lse, int R, void* stream);

/* ------------------------------------------------------------------------------------------
 * The paper's own index form (Sections 4.2-4.4, 5.4, Appendix A): CSR child entries that carry
 * ids of deduplicated per-node matcher rows, tested against per-request attribute rows.
 *   node row   : OR of the rows of every ad below the node (bitmask: W_bm words, Bloom: W_bl words)
 *   bitmask    : passes iff (row AND user_bitmask) == user_bitmask           (Section 4.2)
 *   Bloom      : passes iff for ANY of the request's N_loc location rows q, (q AND row) == q
 *                (Section 4.3); no location row -> no match
 * Child entries follow node order (entry j leads to node j + 1), children of a node are sorted by
 * token.  All pointers device.
 * ---------------------------------------------------------------------------------------- */
typedef struct {
  int32_t V, L, W_bm, W_bl, N_loc, reserved;
  int64_t num_nodes, num_entries;
  const int32_t* node_offsets;      /* [num_nodes + 1]                                   */
  const int32_t* csr_child_nodes;   /* [num_entries]                                     */
  const int16_t* csr_tokens;        /* [num_entries]                                     */
  const int32_t* bitmask_index;     /* [num_entries] row of bitmask_table                */
  const int32_t* bloom_index;       /* [num_entries] row of bloom_table                  */
  const uint64_t* bitmask_table;    /* [n_bitmask_rows][W_bm]                            */
  const uint64_t* bloom_table;      /* [n_bloom_rows][W_bl]                              */
  const uint64_t* user_bitmask;     /* [B][W_bm]                                         */
  const uint64_t* user_blooms;      /* [B][N_loc][W_bl]                                  */
  /* k-way partitioned rows (Section 4.2 "k-way partition", Section 4.4): NULL = one pair of rows per
   * child entry.  Otherwise [num_entries + 1]: entry j owns the partition slots part_offsets[j] ..
   * part_offsets[j+1]-1, bitmask_index / bloom_index are indexed by SLOT (length part_offsets[num_entries]),
   * and an entry is kept iff ANY of its slots passes the bitmask test and the Bloom test. */
  const int32_t* part_offsets;
} grace_gtm_index_t;

/* Host-side builder.  sids host int32 [n_sids][L] sorted and distinct; ads sorted by SID:
 * ad_sid host int64 [n_ads] (index into sids, non-decreasing, every SID has at least one ad),
 * ad_bitmask host uint64 [n_ads][W_bm], ad_bloom host uint64 [n_ads][W_bl].
 * Outputs (host, caller-allocated): node_offsets [num_nodes+1], csr_child_nodes / csr_tokens /
 * bitmask_index / bloom_index [num_nodes-1]; tables of unique rows.  Call once with both table
 * pointers NULL to learn n_bitmask_rows / n_bloom_rows, then again with tables of that size. */
grace_status_t grace_gtm_index_build(const int32_t* sids, int64_t n_sids, int V, int L,
                                     const int64_t* ad_sid, int64_t n_ads, const uint64_t* ad_bitmask,
                                     int W_bm, const uint64_t* ad_bloom, int W_bl,
                                     int32_t* node_offsets, int32_t* csr_child_nodes, int16_t* csr_tokens,
                                     int32_t* bitmask_index, int32_t* bloom_index,
                                     uint64_t* bitmask_table, int64_t* n_bitmask_rows,
                                     uint64_t* bloom_table, int64_t* n_bloom_rows);

/* The same index with k-way partitioned rows (Section 4.2, "k-way partition"): the SIDs below a node are
 * split into groups and one (bitmask, Bloom) pair of union rows is stored per group, in the jagged
 * layout of Section 4.4 (the fixed-width layout of static k-way is the case of equal row lengths).
 *   static  : k_level host int32 [L + 1], k_level[l] = k of the entries that lead to nodes of level l
 *   dynamic : k_level NULL; per node the smallest k in 1..min(k_max, #SIDs below) whose fullest group
 *             has fill (set bits of the pair / its width) <= fill_target, else that upper bound
 * Construction is greedy in SID order: a SID joins the group whose pair has the fewest set bits after
 * OR-ing the SID's rows in (ties: lowest group); empty groups are not stored.
 * part_offsets host [num_nodes] (= entries + 1).  Call once with part_bitmask_index, part_bloom_index and
 * both tables NULL to learn *n_parts and the table sizes, then again with arrays of those sizes. */
grace_status_t grace_gtm_index_build_kway(const int32_t* sids, int64_t n_sids, int V, int L,
                                          const int64_t* ad_sid, int64_t n_ads, const uint64_t* ad_bitmask,
                                          int W_bm, const uint64_t* ad_bloom, int W_bl,
                                          const int32_t* k_level, double fill_target, int k_max,
                                          int32_t* node_offsets, int32_t* csr_child_nodes, int16_t* csr_tokens,
                                          int32_t* part_offsets, int32_t* part_bitmask_index,
                                          int32_t* part_bloom_index, int64_t* n_parts,
                                          uint64_t* bitmask_table, int64_t* n_bitmask_rows,
                                          uint64_t* bloom_table, int64_t* n_bloom_rows);

/* CD + GTM lookup and score add on the index above (the kernel of Section 5.4): for every beam the
 * child-entry range of its node is scanned, bitmask first (stop at the first failing word), Bloom
 * only for entries that pass it (stop at the first location that is contained); the request's rows
 * are staged in shared memory once per thread block.  Outputs as grace_gtm_mask.  V <= 4096,
 * W_bm <= 16, W_bl <= 8, N_loc <= 256. */
grace_status_t grace_gtm_lookup(const float* logp, const float* beam_score, const int32_t* beam_node,
                                const grace_gtm_index_t* index, float* cand, uint64_t* allow_bits,
                                int B, int M, int32_t* d_status, void* stream);

/* grace_beam_update on the CSR form: new_node = the child entry of prev_node[src] whose token matches. */
grace_status_t grace_beam_update_csr(const int32_t* parent, const int32_t* token, const float* score,
                                     const int32_t* prev_node, const uint64_t* prev_key,
                                     const grace_gtm_index_t* index, int32_t* new_node, uint64_t* new_key,
                                     int B, int K, int M_prev, int prefix_len, int32_t* d_status, void* stream);

/* ------------------------------------------------------------------------------------------
 * Beam x codebook top-k (Sections 3.1, 3.3).  Per request b, the K best of cand[b][0..N)
 * under the total order (value descending, flat index ascending); -0.0 == +0.0; -inf takes
 * part like any value.  Outputs are in that order:
 *   out_score fp32, out_flat int32, out_parent = flat / V, out_token = flat % V, each [B][K]
 *   (out_flat / out_parent / out_token may be NULL).
 * Needs a device workspace of grace_beam_topk_workspace_bytes(B, N, K) bytes, 256-byte aligned;
 * its contents on entry do not matter.  1 <= K <= 4096; N < 2^31.  K > N (a beam wider than the
 * candidate set, as step 0 of the paper's fixed schedule (1, 1024, ...) with 512 tokens): all N
 * candidates in order, then K - N dead entries (score -inf, flat = parent = token = 0).
 * ---------------------------------------------------------------------------------------- */
size_t grace_beam_topk_workspace_bytes(int B, int64_t N, int K);
grace_status_t grace_beam_topk(const float* cand, int B, int64_t N, int K, int V,
                               float* out_score, int32_t* out_flat, int32_t* out_parent,
                               int32_t* out_token, void* ws, size_t ws_bytes,
                               int32_t* d_status, void* stream);

/* The same selection with the candidates never materialised: candidate m * V + v of request b is
 *   row_score[r] + (logits[r][v] - row_lse[r])   if bit v of allow_bits[r][] is set,  -inf otherwise,
 * with r = b * M + m: exactly what grace_gtm_mask_logits would have written (same fp32 operations in the
 * same order), so both forms return identical results.  logits fp32 [B*M][V] (V % 64 == 0), allow_bits
 * uint64 [B*M][V/64] and row_lse fp32 [B*M] as produced by grace_gtm_mask_logits with cand = NULL,
 * row_score fp32 [B*M] the beams' prefix scores.  Logits are read only in 16-byte pieces that hold an
 * allowed token, so sparse trie levels cost a pass over the allow bits.  Workspace as grace_beam_topk
 * with N = M * V. */
grace_status_t grace_beam_topk_masked(const float* logits, const uint64_t* allow_bits, const float* row_score,
                                      const float* row_lse, int B, int M, int V, int K,
                                      float* out_score, int32_t* out_flat, int32_t* out_parent,
                                      int32_t* out_token, void* ws, size_t ws_bytes,
                                      int32_t* d_status, void* stream);

/* grace_beam_topk with the scratch memory built into the library (the paper has no counterpart:
 * this exists for callers of this library, not for the method).
 *
 * For callers that cannot allocate device memory where they need the selection -- a plug-in that
 * is handed input and output buffers only, a hot path on which the host framework forbids
 * allocation, a process whose memory pool is already committed -- the per-request headers and
 * candidate lists live in a fixed array inside the library's device image instead of a caller
 * workspace.  Same arguments and results as grace_beam_topk, minus `ws`.
 *   - Limit: B <= grace_beam_topk_static_max_requests() (32; the array is about 2 MB and every GPU
 *     that loads the library holds it until the process exits).  A larger B returns
 *     GRACE_WORKSPACE_TOO_SMALL and launches nothing; K and N limits are those of grace_beam_topk.
 *   - The first call on a device looks up the array's device address (once per device, with that
 *     device current); make that first call before any stream capture.
 *   - The call itself allocates nothing and frees nothing.
 *   - All calls on a device share the one array: calls that may overlap on the GPU (different
 *     streams, or concurrent host threads) race and must be serialised by the caller.  The array
 *     keeps the previous call's contents; the kernels rewrite everything they read, so no clearing
 *     is needed between calls. */
int grace_beam_topk_static_max_requests(void);
grace_status_t grace_beam_topk_static(const float* cand, int B, int64_t N, int K, int V,
                                      float* out_score, int32_t* out_flat, int32_t* out_parent,
                                      int32_t* out_token, int32_t* d_status, void* stream);

/* ------------------------------------------------------------------------------------------
 * Beam-state update after top-k ("rearrangement", Sections 3.3, 4.4).  For new row i of request b:
 *   src = b*M_prev + parent[b][i]
 *   new_key[b*K+i]  = prev_key[src] | (token+1) << 16*prefix_len
 *   new_node[b*K+i] = child(prev_node[src], token)   or -1 if score = -inf or prev_node[src] < 0
 * Only these small arrays move; KV stays where it is.  All device; parent/token/score [B][K].
 * ---------------------------------------------------------------------------------------- */
grace_status_t grace_beam_update(const int32_t* parent, const int32_t* token, const float* score,
                                 const int32_t* prev_node, const uint64_t* prev_key,
                                 const grace_trie_t* trie, int32_t* new_node, uint64_t* new_key,
                                 int B, int K, int M_prev, int prefix_len,
                                 int32_t* d_status, void* stream);

/* ------------------------------------------------------------------------------------------
 * Decoder-layer building blocks used by grace_decode_step (Section 3.2; the paper leaves these
 * GEMMs to a vendor library, Section 5.2 "Kernel fusion").  Exported so each can be checked.
 * ---------------------------------------------------------------------------------------- */

/* y = act(x @ w^T) (+ residual).  x bf16 [M][K] (row stride ldx), w bf16 [N][K] (row stride ldw),
 * fp32 accumulation.  Exactly one of y_bf16 / y_f32 is non-NULL ([M][N], row stride ldy).
 * residual: fp32 [M][N] (row stride ldy) or NULL, added before the store; may alias y_f32.
 * relu != 0 applies max(., 0) before the residual.  K multiple of 64, N multiple of 16;
 * pointers 16-byte aligned, strides multiples of 8 elements. */
grace_status_t grace_linear(const uint16_t* x, int64_t ldx, const uint16_t* w, int64_t ldw,
                            uint16_t* y_bf16, float* y_f32, int64_t ldy, const float* residual,
                            int M, int N, int K, int relu, void* stream);

/* y += x @ w^T with a bf16 residual stream y [M][N] (row stride ldy): the product is accumulated in
 * fp32, rounded to bf16 and added to y in bf16 (large problems: by a TMA add-reduction, y is never read
 * into the SM).  Same shape and alignment rules as grace_linear. */
grace_status_t grace_linear_add_bf16(const uint16_t* x, int64_t ldx, const uint16_t* w, int64_t ldw,
                                     uint16_t* y_inout, int64_t ldy, int M, int N, int K, void* stream);

/* y_f32 = x @ w^T (fp32 output) and, from the same accumulators, the start of every row's log-sum-exp:
 * lse_part fp32 [M][N / 256][2] receives (maximum, sum of e^(y - maximum)) over each 256-column tile of the
 * row.  Large problems only (M >= 1024, N % 256 == 0); otherwise GRACE_UNSUPPORTED_SHAPE. */
grace_status_t grace_linear_f32_lse(const uint16_t* x, int64_t ldx, const uint16_t* w, int64_t ldw,
                                    float* y_f32, int64_t ldy, float* lse_part, int M, int N, int K, void* stream);

/* A LayerNorm folded into the GEMM that consumes it.  With w' = w * gamma (per input feature),
 *   LayerNorm(x) @ w^T  =  rstd * (x @ w'^T)  -  rstd * mean * colsum(w')  +  beta @ w^T,
 * so the GEMM can read the raw bf16 residual stream (no normalised copy is written or read) and finish in its
 * epilogue with two numbers per row and two per column.
 * grace_row_stats_bf16: row_affine fp32 [R][2] = (rstd, -rstd * mean) of x bf16 [R][D] (D % 8 == 0, D <= 2048).
 * grace_linear_folded_ln: y = row_affine[m][0] * (x @ w^T)[m][n] + row_affine[m][1] * col_sum[n] + col_bias[n],
 *   then ReLU if relu; output bf16 (y_bf16) or fp32 (y_f32; with lse_part also the log-sum-exp partials of
 *   grace_linear_f32_lse).  Shapes as grace_linear; col_sum / col_bias fp32 [N], 16-byte aligned.
 *   col_sum may be NULL: the middle term is dropped.  That is exact when every row of x has zero mean, which a
 *   pre-LayerNorm residual stream keeps if everything added into it is centred over the feature axis (embedding
 *   rows minus their mean; output projections minus their mean over the output index): LayerNorm does not see
 *   a per-row shift, so the model computes the same function, and the epilogue then costs one shared-memory
 *   word per column instead of two (the difference between hiding under the next tile's MMAs and not). */
grace_status_t grace_row_stats_bf16(const uint16_t* x, int R, int D, float eps, float* row_affine, void* stream);
grace_status_t grace_linear_folded_ln(const uint16_t* x, int64_t ldx, const uint16_t* w, int64_t ldw,
                                      const float* row_affine, const float* col_sum, const float* col_bias,
                                      uint16_t* y_bf16, float* y_f32, int64_t ldy, float* lse_part,
                                      int M, int N, int K, int relu, void* stream);

/* grace_row_stats_bf16 (over D = K, with eps) followed by grace_linear_folded_ln, as one call: the LayerNorm over
 * the rows of x [M][K] (ldx == K) and the GEMM behind it.  For M >= 1024 and 256 <= N <= 512 with centred rows
 * (col_sum NULL) and no lse_part it is ONE kernel: the row statistics are formed from the GEMM's own operand tiles in shared
 * memory while the tensor cores work on them, so the residual stream is not read a second time; row_affine
 * (device, fp32 [M][2], 8-byte aligned) is then not touched.  Otherwise (wider outputs, where forming the
 * statistics once per 256-column tile costs more than reading the stream once) the statistics kernel runs
 * first, into row_affine.  Other arguments and errors as grace_linear_folded_ln. */
grace_status_t grace_linear_layer_norm(const uint16_t* x, int64_t ldx, const uint16_t* w, int64_t ldw, float eps,
                                       float* row_affine, const float* col_sum, const float* col_bias,
                                       uint16_t* y_bf16, float* y_f32, int64_t ldy, float* lse_part,
                                       int M, int N, int K, int relu, void* stream);

/* The logits GEMM of a constrained decode step (Section 3.1: the constraint is known before the logits are):
 * the products of grace_linear_f32_lse (row_affine NULL) or of grace_linear_layer_norm with lse_part (row_affine
 * = fp32 [M][2] scratch, eps, col_sum / col_bias as there; eps < 0: row_affine already holds the rows' statistics
 * from grace_row_stats_bf16 and is only read), with the same lse_part [M][N / 256][2] over ALL
 * columns, but of the values only those whose bit is set in allow_bits (device, [M][N / 64] words, 16-byte
 * aligned; bit v % 64 of word v / 64 = column v) are stored, at their place in y_f32 [M][ldy]; every other
 * element of y_f32 is left as it was or, if it shares an aligned group of 8 columns (one 32-byte sector) with an
 * allowed one, set to its product as well.  M >= 1024, N % 256 == 0, else GRACE_UNSUPPORTED_SHAPE. */
grace_status_t grace_linear_logits_allowed(const uint16_t* x, int64_t ldx, const uint16_t* w, int64_t ldw, float eps,
                                           float* row_affine, const float* col_sum, const float* col_bias,
                                           const uint64_t* allow_bits, float* y_f32, int64_t ldy, float* lse_part,
                                           int M, int N, int K, void* stream);

/* out bf16 [R][D] = LayerNorm(x fp32 [R][D]) * gamma + beta, eps inside the square root. */
grace_status_t grace_layer_norm(const float* x, const float* gamma, const float* beta,
                                uint16_t* out, int R, int D, float eps, void* stream);

/* x fp32 [R][D] = embed[token[r]] + pos (embed bf16 [V+1][D], pos bf16 [D]); token int32 [R]. */
grace_status_t grace_embed(const int32_t* token, const uint16_t* embed, const uint16_t* pos,
                           float* x, int R, int D, int n_rows_embed, int32_t* d_status, void* stream);

/* The same two with a bf16 residual stream (x bf16 [R][D]; statistics still in fp32; LayerNorm: D % 8 == 0,
 * D <= 2048). */
grace_status_t grace_layer_norm_bf16(const uint16_t* x, const float* gamma, const float* beta,
                                     uint16_t* out, int R, int D, float eps, void* stream);
grace_status_t grace_embed_bf16(const int32_t* token, const uint16_t* embed, const uint16_t* pos,
                                uint16_t* x, int R, int D, int n_rows_embed, int32_t* d_status, void* stream);

/* In place: logits fp32 [R][V] -> log-probabilities (natural log), normalised over all V. */
grace_status_t grace_log_softmax(float* logits, int R, int V, void* stream);

/* Per-layer weights; every matrix is bf16 [out_features][in_features], dense rows. */
typedef struct {
  const float *ln1_g, *ln1_b, *ln2_g, *ln2_b, *ln3_g, *ln3_b;
  const uint16_t *w_qkv;   /* [3*H*d_h][d_model]  rows ordered (q|k|v, head, i) */
  const uint16_t *w_o;     /* [d_model][H*d_h] */
  const uint16_t *w_qc;    /* [H*d_h][d_model] */
  const uint16_t *w_oc;    /* [d_model][H*d_h] */
  const uint16_t *w_1;     /* [d_ffn][d_model] */
  const uint16_t *w_2;     /* [d_model][d_ffn] */
  const uint16_t *k_cross, *v_cross;   /* [B][T_ctx][H][d_h]: as the once-per-request projection
                                          GEMM of the encoder output writes them (Section 3.2) */
  uint16_t *k_cache, *v_cache;         /* [L][R_max][H][d_h]; unused (may be NULL) when qkv_slabs is set */
  /* With grace_decoder_t.ln_folded: w_qkv, w_qc, w_1 already carry the gain of the LayerNorm in front of
   * them (w[n][k] * gamma[k], rounded to bf16) and these hold, per output feature n, the sum over k of that
   * matrix (cs_*) and the sum over k of beta[k] * (unfolded) w[n][k] (cb_*), fp32 [out_features]. */
  const float *cs_qkv, *cb_qkv, *cs_qc, *cb_qc, *cs_1, *cb_1;
  /* NULL, or [L][R_max][3*H*d_h]: the QKV projection of step t is written into slab t and kept, and the
   * self-attention reads its cache from the K and V thirds of the slabs (grace_self_attn_inplace). */
  uint16_t *qkv_slabs;
} grace_layer_t;

#define GRACE_MAX_LAYERS 16
#define GRACE_MAX_STEPS 8

/* Everything one decode step reads and writes.  A plain struct of caller-owned device buffers
 * (host struct, passed by pointer, read during the call only). */
typedef struct {
  int32_t B, n_layers, d_model, H, d_h, d_ffn, V, L, T_ctx;
  int32_t beam_sizes[GRACE_MAX_STEPS + 1]; /* M_0 .. M_{L-1}, then the final K at index L  */
  int64_t R_max;                           /* B * max beam size                             */
  float ln_eps;
  grace_layer_t layers[GRACE_MAX_LAYERS];
  const uint16_t *embed;      /* [V+1][d_model], row V = start token */
  const uint16_t *pos;        /* [L][d_model]                        */
  const float *lnf_g, *lnf_b;
  const uint16_t *w_out;      /* [V][d_model]                        */
  grace_trie_t trie;
  grace_matcher_t matcher;
  /* beam state, double-buffered by step parity: index (t & 1) is read, ((t+1) & 1) written */
  int32_t *token[2];          /* [R_max] input token of each row                          */
  float *score[2];            /* [R_max]                                                  */
  int32_t *node[2];           /* [R_max]                                                  */
  uint64_t *key[2];           /* [R_max]                                                  */
  int32_t *parents;           /* [L+1][R_max]; slab t+1 is written by step t               */
  int32_t *out_flat;          /* [R_max] scratch for the selected flat indices             */
  /* activations (scratch) */
  float *x;                   /* [R_max][d_model] fp32 residual stream, or NULL ...        */
  uint16_t *x_bf16;           /* ... then [R_max][d_model] bf16 residual stream            */
  uint16_t *h;                /* [R_max][max(d_model, d_ffn)]                             */
  uint16_t *qkv;              /* [R_max][max(3*H*d_h, d_ffn)]: qkv, cross-q, FFN hidden     */
  uint16_t *attn;             /* [R_max][H*d_h]                                            */
  float *logp;                /* [R_max][V] log-probabilities; raw logits when row_lse is set */
  float *row_lse;             /* NULL, or [R_max]: fuse log-softmax into the mask kernel; the
                                 per-row log-sum-exp lands here (0 for dead rows)            */
  float *cand;                /* [R_max][V] masked scores; may be the same buffer as logp  */
  uint64_t *allow_bits;       /* NULL, or [R_max][V/64] (needs row_lse): from step masked_from_step on the
                                 mask kernel writes only these bits and the top-k reads the logits through
                                 them (cheaper where few tokens per row survive; where a fifth of the row
                                 survives and the whole logits tensor is written anyway, materialised
                                 candidates are faster); earlier steps use cand                          */
  int32_t masked_from_step;   /* first step (0-based) that takes the allow-bits path                   */
  int32_t logits_allowed_only; /* != 0 (needs allow_bits, row_lse, lse_part): on the allow-bits steps of large
                                 width the constraint runs BEFORE the logits GEMM, which then stores only the
                                 allowed logits; logp holds valid values only where a token is allowed */
  float *lse_part;            /* NULL, or [R_max][V/256][2] (needs row_lse, V % 256 == 0): the logits GEMM
                                 leaves per-tile log-sum-exp partials and the mask kernel merges them     */
  /* LayerNorms folded into the GEMMs behind them (bf16 residual stream only): NULL, or [R_max][2] scratch
     for the row statistics; then w_qkv / w_qc / w_1 / w_out carry the gains and cb_* are set; cs_* are set
     too unless the caller keeps the stream's rows at zero mean (see grace_linear_folded_ln). */
  float *row_affine;
  const float *cs_out, *cb_out;   /* [V] for the output head (final LayerNorm)                         */
  void *topk_ws; size_t topk_ws_bytes;
  int32_t *d_status;
} grace_decoder_t;

/* Host-only consistency check of a decoder struct (null pointers, shape limits). */
grace_status_t grace_decoder_validate(const grace_decoder_t* dec);

/* Start state of a decode loop (Section 3.3: M_0 = 1): for each of the B requests, input token =
 * start token (V), score 0, node = root, key 0, written to state buffers [0]; *d_status = 0. */
grace_status_t grace_decode_begin(const grace_decoder_t* dec, void* stream);

/* Step t (0-based) of the decode loop (Sections 3.1-3.3): embed the rows' input tokens, run the
 * decoder layers (self-attention with cache write, cross-attention, feed-forward), logits,
 * log-softmax, CD+GTM mask with score add, top-k of beam_sizes[t+1] per request, state update.
 * Reads state buffers [t & 1], writes [(t+1) & 1] and parents slab t+1. */
grace_status_t grace_decode_step(const grace_decoder_t* dec, int t, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* GRACE_H_ */
