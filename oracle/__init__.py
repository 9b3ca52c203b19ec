"""CPU oracle for the LASER Draft-Then-Verify loop (arXiv 2408.05676).

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, obviously-correct
restatement of what the decoding loop computes, written from the paper:

* ``retrieval`` - Retrieve(D, tail, K) of Eq. 5 / Section 3.3 as a linear scan
  of the group's token array (equivalent to the per-group trie of Section 3.2),
* ``forward``   - the target model's verify forward of Eq. 3 / Eq. 6 for a
  Llama-style decoder in fp64 (bf16 weights, bf16 K/V cache),
* ``accept``    - greedy verification (Eq. 4) and Relaxed Verification (Eq. 8)
  plus the ablation variants of Section 4.3.2, in fp64,
* ``generate``  - the Draft-Then-Verify loop of Section 2.1 and plain
  autoregressive greedy decoding (Eq. 1).

It shares no code with the CUDA library, never imports it, and must only be
used by the tests, by the smoke check and by the benchmark's CPU baseline.
Every function is pinned by tests that run without a GPU (hand-worked
examples, closed forms, brute force, invariants); no function is left
"parity unpinned".
"""
