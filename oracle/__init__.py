"""CPU oracle for the compressed linear-operator step (TEST INFRASTRUCTURE ONLY).

This package is a plain, slow, double-precision restatement of what the paper's
compressed linear operator computes (Definition 3.1 and Section 4), plus the
frozen "Gaussian v1" sketch generator.  It exists so that the CUDA library can
be checked against something written independently of it.

Rules this package keeps:
  * it shares no code, tables, constants generators or helpers with the CUDA
    path, and imports nothing from ``paper_2605_01255_b200``;
  * only ``tests/``, ``__graft_entry__.smoke()`` and the ``cpu_baseline`` /
    ``--impl reference`` legs of ``bench.py`` may import it;
  * it is never a fallback for the product: the product fails loudly when its
    CUDA library is missing.

Parity status: every function in ``oracle.sketch``, ``oracle.linear`` and ``oracle.optimizer`` is
pinned by the CPU tests (known-answer vectors, closed forms, brute force,
invariants).  What stays *parity unpinned* is anything that needs the paper's
trained models or datasets (accuracy, loss curves, absolute values of
Table A1, memory in GB of a real fine-tuning run); none of that is computed
here.
"""
