"""fp64 CPU oracle of the MoDA attention operator -- TEST INFRASTRUCTURE ONLY.

Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU-baseline / ``--impl reference``
legs of ``bench.py`` may import this package.  The product package never does, and this
package never imports the product package: the two share no code.
"""
