"""fp64 CPU oracle for the DiTango selective attention-state path.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline / reference legs of the benchmark.  The product path never imports
it, and it never imports the product path.
"""
