"""fp64 CPU oracle for the matrix-form minibatch-SGD training step.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this
directory; only the test-suite, the smoke check and the CPU-baseline leg of
the benchmark do.  It shares no code with the CUDA path.

Modules
  mbd_oracle  plain numpy/fp64 statement of forward, loss, backprop, SGD
              update (Section 1, Eq. 1; Appendix A.1/A.2), un-blocked and
              blocked over a P_r x P_c grid, plus the 3x3 convolution used by
              the domain-parallel configuration (Section 2.2, Eq. 7).
  brute       scalar pure-Python loop nests of the same definitions, for tiny
              shapes only; pins mbd_oracle.
  comm_words  bandwidth terms of Eq. 3, 4, 7, 8, 9 as exact integers.

Parity status: every function here is pinned by tests run with
`-m "not gpu"` (finite differences, brute force, adjoint identities, closed
forms, blocking invariance).  The simulated speed-ups the paper quotes in
Section 3 are not reproduced here (they need a layer table and timings the
paper only plots): parity unpinned for those, and nothing computes them.
"""
