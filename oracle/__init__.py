"""CPU oracle for the chunked, arena-placed DiT block -- TEST INFRASTRUCTURE ONLY.

A plain, slow, float64 statement of what the hot path computes, written from the
paper (static-layout section, Algorithm 1; the "only as much mitigation as
needed" selection rule) and, for the block arithmetic the paper does not spell
out, from the standard operator definitions listed in the repository's design
notes.  It shares no code with the CUDA library and must never be imported by
the product package; only the tests, the smoke check and the benchmark's CPU
baseline leg may use it.

  oracle.block  -- adaLN / QKV / RMSNorm / RoPE / attention / FFN in float64
  oracle.trace  -- tensor lifetimes of the block template for a chunk count
  oracle.arena  -- Algorithm 1 (size-descending best-fit layout), max-live,
                   and the smallest chunk count that fits a byte budget

Parity status: the planner parts (trace, layout, chunk search) are pinned by
closed forms, hand-worked layouts and brute force; the block arithmetic is
pinned by brute-force attention, softmax/LN/RoPE invariants, special weight
settings with known answers and an independent torch-float64 restatement.
Which operator definitions apply (adaLN form, RoPE pairing, epsilons, ...) is
a reading the paper does not fix: on that point parity is "unpinned".
"""
