"""CPU oracle for the mixed-batch step (test infrastructure only).

This package is TEST INFRASTRUCTURE. It is a plain, slow, obviously-correct
CPU statement of what one heterogeneous-batching forward step must produce.
Only the tests, the smoke check and the benchmark's CPU-baseline leg may
import it; the product package never does, and nothing here imports the
product package or its CUDA library.

Modules
-------
transformer  the plain definition: whole-sequence forward, single-pass
             embedding, full-recompute greedy generation (Section 2.1 of the
             paper for the three request kinds, Section 3.1 "forward ...
             identical across request types").
method       the method restated step by step: chunked execution over a
             growing dense K/V list, the incremental pooler of Section 3.3
             (Eq. 1-2, and the positional heads), decode over cached K/V, and
             the integer bookkeeping (page slot map, pool counters).  Used to
             brute-force the method's invariants against `transformer`.
scalar       the same forward in pure Python loops, for tiny shapes only;
             pins the array code of `transformer` against index mistakes.

Parity status: every function is pinned by the CPU test-suite (library
routines, closed forms, invariants, brute force); nothing is "parity
unpinned".
"""
