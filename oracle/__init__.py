"""CPU oracle for the tree-packed linear-attention path.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline legs may import this
package; the product (the CUDA library and its binding) never does, and this package
never imports the product.

Pins (see tests/test_oracle_*.py, tests/test_plan_oracle.py):
  * la_oracle   -- token recurrence fwd/bwd: closed forms (cumulative sum, geometric
                   series), the dense decay-masked matmul form, central finite differences,
                   fp64 autograd of the dense form, equality with a depth-first compact
                   evaluation of the tree, invariance to how dO is split over copies.
  * plan_oracle -- Algorithm 1: brute-force minimum call counts on tiny trees, the worked
                   examples of Figs. 1-3, the strict boundary cases, the replay total of
                   Eq. 15, fp64 execution of the plan against la_oracle.
  * logp_oracle -- Eqs. 17/19/20 (mapped log-probability, its gradient, multiplicity): uniform
                   and two-word closed forms, torch log_softmax + autograd on the expanded
                   rows, central finite differences, zero row sums and shift invariance,
                   hand-counted positions of the five-node tree.
  * conv_oracle -- tree-aware causal convolution (Section 4.2): torch conv1d on every expanded
                   trajectory, autograd through the expansion, identity/shift filters on the
                   five-node tree, central differences.
  * attn_oracle -- full attention on compact tokens (Section 3.4, Eqs. 21-22): torch causal
                   scaled_dot_product_attention on every expanded trajectory with autograd
                   through the expansion, the bottom-right mask of a branch view, equal-keys
                   closed form, central differences.
  * mb_oracle   -- microbatch planning (Section 3.2): Eq. 5 / Eq. 6 / the range-minimum LCP rule
                   against the brute-force trie count, hand-counted costs of the five-node tree,
                   the slot-schedule rule; the search itself has no closed form and is checked
                   for validity and against brute force over contiguous cuts.
  * Appendix planning cases I-III: parity unpinned (the trees' token counts were only in
                   the figures); only the printed totals are checked for self-consistency.
"""
