"""Seeded synthetic inputs (shapes and value recipes of the benchmark configurations).

Used by the tests, bench.py and the smoke test; holds none of the method's arithmetic and is not
part of the library.
"""
