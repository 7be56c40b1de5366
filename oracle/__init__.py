"""CPU oracle for the TS + TAB-Q codec.

Test infrastructure only: nothing under this package is part of the product path.
Only the tests, the smoke check and the benchmark's CPU-baseline leg import it.
"""
