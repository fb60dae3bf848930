"""CPU oracle for the chunk-pipelined reduce / broadcast over an object store.

TEST INFRASTRUCTURE ONLY.  Nothing here is part of the product: only ``tests/``, the
smoke check and the benchmark's CPU-baseline leg may import it.  It is written from the
paper (Hoplite, arXiv 2002.05814, Section 3) in plain Python + numpy, shares no code
with the CUDA library and never imports it.

What each module restates:

* ``reduce_tree``    -- Section 3.4.2: d-ary reduce tree, arrival-order placement by the
                        generalised in-order traversal, k-of-m selection; Section 3.5.2:
                        removal of a failed node, replacement by the next ready source,
                        clearing of the ancestors' partial results.
* ``broadcast_tree`` -- Section 3.4.1: receiver-driven broadcast through the object
                        directory (one location per query, complete copies preferred,
                        sender removed while sending); Section 3.5.1: failover of a
                        receiver whose sender failed, without cyclic dependencies.
* ``values``         -- the plain definitions the method must reach: the reduce of the
                        selected objects (in tree association order for fp32 bit patterns,
                        and left to right in fp64 as the brute-force check) and
                        byte-identical broadcast copies.
* ``store``          -- Sections 3.1-3.3: object directory entries (size, locations with a
                        partial/complete bit, refined to a chunk prefix), Put / Get /
                        Reduce / Delete (Table 1) driven by a timeline of events.

Parity status of the parts the paper does not fix:
the tree after a failure that leaves fewer live sources than requested ("shrink"), the
broadcast sender choice for more than one send slot per location, the order in which the
orphans of one failure ask again, and the way a prefix crosses dtypes in composed collectives
are build-defined readings.  Each is held to a hand-worked example under ``tests/golden/``
(``reduce_shrink_example``, ``broadcast_two_slots_example``, ``broadcast_orphans_example``,
``composition_cross_dtype``; ``tests/test_golden_rules.py``) besides the invariants and
brute-force value checks in ``tests/test_oracle_*.py``.  The order in which SEVERAL waiting receivers would be served is not pinned because it cannot be
observed: at most one receiver ever waits (a second one could fetch from the first), which
``tests/test_oracle_broadcast.py`` checks over random timelines.
"""
