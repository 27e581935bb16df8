"""CPU oracle for the hierarchical, load-weighted gradient synchronisation.

Test infrastructure only: imported by tests, the smoke check and the bench's
CPU-baseline leg.  Independent of the CUDA library (no shared code either way).
"""
