"""CPU oracle for two-dimensional KV-cache migration. TEST INFRASTRUCTURE ONLY.

Nothing in the product package imports this directory; only tests, the smoke check and the benchmark's
CPU-baseline / reference legs do.
"""
