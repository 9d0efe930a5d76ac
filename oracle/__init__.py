"""CPU oracle for the Prof-K hot path.  TEST INFRASTRUCTURE ONLY.

Everything in this package is a plain, slow, CPU-only restatement of what the
GPU path has to compute, written from the paper so that a reader can check it
against the paper by eye.  It exists to check the CUDA library; it is not a
fallback for it.  Only the tests, the smoke check and the CPU-baseline leg of
the benchmark may import it.  It shares no code with the CUDA sources: the
order-preserving key transform, the parameter formulas, the binomial / hyper-
geometric tails and the Philox generator are each written out a second time
here, on top of NumPy / SciPy.

Modules
-------
topk      exact top-k by definition (full sort, tie rule "value descending,
          index ascending"), a brute-force twin for tiny inputs, and an O(N)
          checker of a claimed answer.                    (Section 3, problem setup)
plan      Algorithm 1 literally, the equations it is built from, and the
          guarded plan the library returns.               (Section 4, Algorithm 1)
rank_law  Lemma 1 (negative hypergeometric law of the threshold rank) and the
          exact failure probabilities that follow from it.
philox    Philox4x32-10 and the stratified sample-index recipe.
stages    the four stages (sample, threshold, filter, refine/fallback) run
          literally on a NumPy array.                     (Section 3)
mc        Monte Carlo estimates of the two failure events.

Parity pins: see each module's header.  For `plan.plan_guarded` in relaxed-recall
mode (recall < 1) the paper prints no formula; that mode is pinned by Lemma 1's
exact tail for the accepted count, minimality of the rank and a Monte Carlo of
the two failure events (tests/test_oracle_plan.py, tests/test_oracle_mc.py).
"""
