"""fp64 CPU oracle for the Q-Delta hot path.

TEST INFRASTRUCTURE ONLY.  Only the test-suite, the smoke check and the
benchmark's CPU-baseline leg may import this package.  The CUDA library and its
Python binding never do, and the two share no code.

Contents
--------
``recurrence``      ctypes front-end of ``qdelta_oracle.c``: the token-by-token
                    recurrence (Section 3.3.1, gated update rule and read-out)
                    and its hand-written reverse pass.  This is THE oracle.
``chunkwise_form``  a separately written numpy fp64 chunkwise-parallel form
                    (Section 3.3.2, chunk expansion / extended WY / UT
                    transform) and its chunk-level backward; used only to
                    cross-check the recurrence oracle.
``build``           compiles the C file with gcc.

Pins (what the oracle is checked against, see tests/test_oracle_*.py): the
closed form of one step and the three printed forms of the rule; reduction to
an independently coded (gated) delta rule at lambda = 0; the beta = 0 closed
form; the exact error identity in the proof of Lemma 1 and the per-step
inequality of Theorem 1; the explicit product of transition matrices of the
chunk expansion; the value-span decomposition of Section 3.1; the extended WY
identity; chunk-size and segment invariance; central finite differences and a
dot-product (adjoint) test for the reverse pass.  No function is unpinned.
"""
