"""CPU oracle for Overlap-Local-SGD (Wang, Liang, Joshi, arXiv 2002.09539).

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, fp64 restatement of
what the paper's Section 2 ("Proposed Algorithm") computes, written so that it
can be checked against the paper by eye.  It is imported by the test-suite, by
the smoke check and by the CPU-baseline leg of the benchmark, and by nothing
else: the CUDA library never calls it and shares no code, table or constant
generator with it.

Modules
-------
philox      Philox4x32-10 counter-based generator (Salmon et al., SC'11).
sampling    minibatch index rule xi_k^(i) ~ D_i and the worker -> class-pair
            partition table.
models      loss and gradient of the three model families, fp64.
olsgd       the iteration itself: Eq. 3 (local step), Eq. 4 (pull-back),
            Eq. 5 (anchor refresh), Eq. 10-11 (anchor momentum), and the
            matrix form Eq. 8-9 as a second, independent statement.

Parity status: every function here is pinned by tests/test_oracle_*.py against
something other than itself (published known-answer vectors, closed-form
recursions, finite differences, the matrix form, brute force on tiny inputs).
The accuracy numbers of the paper's Tables 1-2 are "parity unpinned": they need
CIFAR-10 and ResNet-18, which are out of scope.
"""
