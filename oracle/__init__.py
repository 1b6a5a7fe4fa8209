"""CPU oracle for tree-decode attention over prefix-shared KV.  TEST INFRASTRUCTURE ONLY.

Nothing here is part of the product: the CUDA library never imports, links or calls
this package, and this package never imports the library.  Only the test-suite, the
smoke check and the benchmark's CPU-baseline leg use it.

What it defines (and where each definition comes from):

* ``tree_attention.tree_decode_attention`` - the exact result the fast path must reach:
  for every live leaf, plain softmax attention of its one query over the concatenated
  K/V of its root-to-leaf path.  The paper gives no attention formula; it only states
  that trajectories sharing a node share that node's KV cache (Section 4.1) and that
  decoding is bound by loading that KV (Sections 1 and 3).  The result is therefore
  the textbook definition softmax(q K^T / sqrt(d)) V, evaluated in fp64 on each
  leaf's fully materialised path.  Pinned by tests/test_oracle_pins.py (single-token
  tree, independent sequences vs. a library attention routine, node splitting, brute
  force, closed forms, permutation invariance, convexity, duplicate leaves).

* ``tree_attention.tree_prefill_attention`` - the same definition for the tokens of a newly
  generated step (what scoring or prefilling a step computes): ancestors whole, the own step up
  to a per-query limit, i.e. causal inside the step.  Pinned by a library causal-attention
  routine on a root step, by the decode oracle on truncated trees, and by an explicit mask.

* ``tree_attention.merge_partials`` - the log-sum-exp combination of per-node softmax
  partials, written out in fp64 only so that tests can show it equals the direct
  definition.  The direct function above never calls it.

* ``flatten.ReferenceFlattener`` - the canonical page/segment/group tables for a tree,
  under the page-assignment and ordering rules stated in its docstring.  Pinned by
  invariants (pages partition, group/path duality, hand-worked small tree in
  tests/golden/).

* ``selection`` - the selection step the paper is about (Section 4, Appendix B): REBASE weights
  (Eq. 1 / Eq. 3), the objective of Eq. 4 and its maximiser by enumeration of leaf subsets.
  Pinned by tests/test_oracle_selection.py (weights and objective values worked by hand from
  the equations, the lambda = 0 and large-lambda closed forms, monotonicity, relabelling).

Numerical parity with values printed in the paper is unpinned by construction: the
paper prints none for this path.  Parity is to the definition.
"""
