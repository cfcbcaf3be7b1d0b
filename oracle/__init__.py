"""CPU oracle (test infrastructure only).  See tq_oracle.c for what it implements.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
"""
