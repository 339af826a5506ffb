"""CPU oracle for the retention-based KV eviction decode path (test infrastructure only).

Nothing in the product package imports this directory; only the tests, the smoke
check and the benchmark's CPU-baseline leg do.
"""
