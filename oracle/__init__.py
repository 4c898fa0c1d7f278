"""CPU oracle for exact ragged Top-K selection (test infrastructure only).

This package is the checker, not the product.  It is imported only by the test
suite, by the smoke check and by the benchmark's CPU-baseline / reference arm.
It shares no code with the CUDA library and never imports it; the CUDA library
and its Python binding never import this package.

Modules
-------
topk_definition : the plain definition of the operator (stable sort per row)
                  written with numpy, fp32 bit patterns handled as integers.
native          : the same definition in C++ (std::stable_sort, OpenMP over
                  rows) plus an independent std::nth_element selector, built by
                  ``oracle.build`` with g++ and reached through ctypes.
sampled_steps   : the paper's three phases (Section 4.2-4.4) restated step by
                  step in numpy, returning both the selected set and the
                  intermediate quantities (tau_0, tau_1, C(tau_0), route).

Parity pins (tests/test_oracle_*.py): rank-counting brute force on tiny rows,
closed forms for structured rows, the exactness criterion of Section 6.1, the
finite-population order statistic of Section 3.2, torch.sort as an unrelated
library routine.  No function here is "parity unpinned".
"""
