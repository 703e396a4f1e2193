"""CPU oracle for the quantized backward pass of arXiv 2407.12637.

TEST INFRASTRUCTURE.  Only tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; the CUDA library and its Python
binding never do.  `oracle.ref` wraps the plain-C implementation
(`lbt_oracle.c`), `oracle.analysis` holds the sort-based error metrics of
Sec. 3.2 / 3.3 (Eq. 5-10) in binary64 numpy.
"""
