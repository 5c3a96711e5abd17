"""Test infrastructure: slow fp64 CPU statement of pdADMM-G / pdADMM-G-Q.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this package.  It shares no code with the CUDA path.
"""
