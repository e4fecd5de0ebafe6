"""TEST INFRASTRUCTURE: fp64 CPU oracle of the coalesced attention engine.

Only tests, ``__graft_entry__.smoke()`` and ``bench.py``'s cpu_baseline / reference arm
may import this package.  It shares no code with the CUDA path and must never be used
by it.
"""
