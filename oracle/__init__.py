"""CPU oracle for the QuEST quantized-linear forward path.

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by ``__graft_entry__.smoke()`` and by the
``cpu_baseline`` / ``--impl reference`` legs of ``bench.py``.  Nothing in the product package
imports it, and it imports nothing from the product package.
"""
