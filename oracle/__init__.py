"""CPU oracle of the Sailor plan simulator and exhaustive search — TEST INFRASTRUCTURE ONLY.

Imported by the tests, the smoke check and the benchmark's CPU-baseline leg; never by the
CUDA package.
"""
