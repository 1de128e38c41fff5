"""CPU oracle for the SFDA hot path -- TEST INFRASTRUCTURE ONLY.

Only ``tests/``, ``__graft_entry__.smoke()`` and the ``cpu_baseline`` /
``--impl reference`` legs of ``bench.py`` may import this package.  The CUDA
library and its Python binding never do, and this package never imports them:
the two share no code, tables or helpers.

Contents
--------
``recurrence``   per-token recurrence in complex double (C, ``sfda_recurrence.c``):
                 the definition of the layer (Section 3, Eq. "sfda").
``chunk_wy``     naive chunked path in numpy complex128 that takes the steps of
                 Algorithm 1 (constructive chunk-WY summary), Theorem "Exact
                 affine chunk transfer" and Theorem "Prefix outputs inside a
                 chunk" literally, one token at a time.
``bookkeeping``  integer side: chunk plan and the quantised cumulative phase.

Every function is pinned by ``tests/test_oracle_pins.py`` against facts that do
not come from this package (dense brute force, closed forms, special cases that
reduce to independently written routines, invariants the paper proves).
"""
