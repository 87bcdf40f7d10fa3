"""CPU oracle for the Hop hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 restatement of what the paper (arXiv 1902.01064) defines, written
from the paper alone.  It shares no code with the CUDA library and imports nothing from
it; only the tests, the smoke check and the benchmark's CPU-baseline leg may use it.

  protocol.py  queue protocol of Figs. alg1-alg4 and Section 5, tick by tick, with literal
               FIFO update queues tagged (iter, w_id) and literal token queues -> trace
  update.py    Reduce / Apply rules (Fig. alg0, Fig. alg4 Reduce, Eq. 2), hinge SVM
               gradient, momentum, all in float64
  philox.py    Philox4x32-10 counter generator + Box-Muller for the synthetic gradients

Parity pins (tests/test_oracle_*.py): Theorems 1 and 2, the token-count identity, Table 1,
the prose examples of Sections 3.4, 3.5, 4.2, a bounded-staleness example worked by hand from
Section 4.4 / Eq. 2 / Fig. alg3, max-plus recurrences of the start and finish times (parallel and
serial approach), Eq. 1 / Eq. 2 closed forms, reduction to a library matmul, all-reduce average on a
complete graph, conservation / convex-hull properties, finite differences of the hinge loss,
torch.optim.SGD for momentum and weight decay, published Philox known answers.
tests/test_oracle_mutations.py plants single-line mistakes here and checks that these pins notice.

Parity unpinned by the paper (fixed by this build's stated readings, guarded only by
invariants and exhaustive agreement between two independent implementations): the hybrid
backup+staleness Recv rule (with backup_exact under NEW_ONLY: kept set first, then only what is new),
the same-tick ordering rule, the skip trigger, the weight of a jumping worker's own parameters,
the default max_ig.
"""
