"""CPU float64 oracle for LoopSpec (test infrastructure, not product code).

A plain, slow, from-the-paper implementation of the looped language model,
vanilla decoding and the LoopSpec scheduler / gate / cascade verification.
Only tests, the smoke check and the benchmark's CPU-baseline leg may import
it; it shares no code with the CUDA path.

Parity status of what lives here:
  * model forward, depth-indexed KV  : pinned (cache-free library forward; for the prelude / recurrent / coda layout
    also the adapter on [state; prelude output], the prelude cache and every readout depth's coda cache)
  * residual operator, cascade rule  : pinned (exact enumeration, chi-square, Thm 1)
  * top-k / top-p filter, masked second proposal: pinned (definition on small
    cases, exact enumeration of the output law)
  * envelope fit (Sec. 4.1)           : pinned (closed form on power-law data)
  * Philox4x32-10                    : pinned (published known-answer vectors)
  * closed-form depths, branch bound : pinned (values printed in the paper)
  * scheduler (Algorithm 1)          : pinned (losslessness, commit-gap schedule)
  * gamma, TV profile log            : pinned (hand values on scripted timelines / hand-made distributions)
  * sampled token streams / gamma on the large shapes: parity unpinned by the
    paper (it prints no token-level example); fixed only by the checks above.
"""
