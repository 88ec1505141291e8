"""CPU oracle for the SwiLA recurrence: test infrastructure only.

Nothing under this package is part of the product path.  It may be imported only by
the tests, by the smoke check, and by the benchmark's cpu_baseline / reference arm.
It imports nothing from the CUDA package.
"""
