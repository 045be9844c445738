"""fp64 CPU oracle for the SSD layer and the MA-GC schedule. TEST INFRASTRUCTURE ONLY.

Nothing in the product package imports this; only tests/, the smoke check and the
bench's CPU-baseline leg do.
"""
