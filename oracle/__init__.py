"""CPU oracle for the GRACE decode step.  TEST INFRASTRUCTURE ONLY.

A plain, slow numpy restatement (fp64 unless noted) of what the decode step
computes, written from the paper's definitions.  It shares no code with the
CUDA library and never imports it.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this package; the product path never
does.

Pin status (what each function is checked against, besides itself):
  attention.cross_attn / self_attn  pinned: per-row textbook SDPA, closed forms
                                    (T=1, equal keys), permutation invariance,
                                    the Section 5.2 block-diagonal example,
                                    block-table / dense-copy equivalence.
  sid_trie.SidTrie                  pinned: set-of-prefixes brute force.
  matchers.* (paper forms)          pinned: the Section 4.2 worked example,
                                    no-false-negative property of OR-unions.
  matchers.PrefixBloom, node_eligibility  pinned: brute-force membership,
                                    analytic false-positive rate.
  kway.* (k-way partitioned rows)   pinned: k = 1 equals the union index, the
                                    Section 4.2 example is filtered with two
                                    groups, ad-level eligibility never lost,
                                    one group per SID is exact, greedy rule by
                                    hand.
  gtm.gtm_mask                      pinned: brute force over all (row, token).
  topk.beam_topk                    pinned: python sorted() with the same key.
  decoder.beam_search               pinned: exhaustive enumeration on tiny
                                    catalogs; score monotonicity invariants.
  decoder.decoder_forward           PARITY UNPINNED against the paper: the
                                    paper gives layer count and head shape but
                                    not norm placement, activation, biases or
                                    position encoding.  Only self-consistency
                                    checks exist (LayerNorm moments, logsumexp
                                    of log-probs = 0, fp32 vs fp64 agreement).
"""
