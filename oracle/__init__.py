"""CPU oracle for the packed low-bit convolution path (test infrastructure only).

Nothing in the product package imports this.  Only ``tests/``, the smoke check
and the benchmark's CPU-baseline leg may use it.  Three parts:

* ``direct``        - the plain definitions (Eq. 2-4, Eq. 16, shift-and-clamp,
                      2x2 max-pool) in int64, C compiled with gcc.
* ``packed_model``  - the paper's own steps (Eq. 5 pack, one wide multiply,
                      Theorem 2 overlap-add, Eq. 29 split, Theorem 3 row
                      mapping) in Python big integers, for small cases.
* ``plan``          - Eq. 6-8, the three guard-bit rules, Eq. 24 and the
                      Algorithm 1 search, by brute force.
"""
