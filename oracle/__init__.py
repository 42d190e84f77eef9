"""CPU oracle for the grouped aggregate + update path.

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
CPU-baseline / reference legs of ``bench.py``.  The product package never
imports it, and it never imports the product package.
"""
