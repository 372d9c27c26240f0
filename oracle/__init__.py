"""CPU oracle for the PTQTP dual-trit-plane linear layer.  TEST INFRASTRUCTURE ONLY.

This package is a plain, slow, fp64 restatement of what the method computes:

* ``oracle.layer``      -- the decode-time layer product
                           y = alpha1 (.) (T1 x) + alpha2 (.) (T2 x) with group-wise
                           scales (Eq. 1-2 with the grouping of the "Batch Processing"
                           paragraph of Sec. 2.3).
* ``oracle.decompose``  -- the progressive trit-plane decomposition (Algorithm 1 for the
                           group structure and stopping rule, Algorithm 2 and Appendix C
                           for the inner formulas).
* ``oracle.bruteforce`` -- exhaustive 9^K enumerations used to pin the T-step and to
                           bound the quality of the alternating scheme on tiny rows.
* ``oracle.packed_format`` -- a byte-level reader/writer of the packed-plane format,
                           written from the format's description, used to check the
                           GPU pack/unpack kernels.
* ``oracle/c``          -- the same layer product and decomposition as plain C loops
                           (timed as the CPU baseline, and fast enough for whole
                           LLaMA-shaped matrices).

Nothing here is imported, linked or executed by the product path.  Only the tests, the
smoke check and the benchmark's CPU-baseline leg may use it.  It shares no code with the
CUDA library: no headers, tables, helpers or constants.

Pins (what fixes each function, beyond itself) live in ``tests/test_oracle_*.py``.
Parity unpinned: the *magnitude* of the reconstruction error of ``decompose`` on
Gaussian weights (the paper prints perplexities only); everything else is pinned.
"""
