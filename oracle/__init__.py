"""TEST INFRASTRUCTURE — not part of the product.

Slow, plain fp64 CPU statement of the static-tree verification path, written
from the paper (Sections 3.1 and 3.2).  Only ``tests/``, the smoke check and
the benchmark's CPU-baseline leg may import this package; the product never
does, and this package never imports the product.
"""
