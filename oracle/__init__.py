"""TEST INFRASTRUCTURE: slow, plain CPU oracle for the asymmetry-aware persistent GEMM path.

Only ``tests/``, ``__graft_entry__.smoke()`` and the ``cpu_baseline`` / ``--impl reference``
legs of ``bench.py`` may import this package.  It shares no code with the CUDA path and
never imports it.
"""
