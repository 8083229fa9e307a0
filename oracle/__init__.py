"""CPU oracle: test infrastructure, not product code.

Only the tests, the smoke check and the benchmark's CPU-baseline leg import this package.  It holds
a plain fp64 statement of what the attention forward pass computes, of the paper's tile schedule
(persistent CTAs with cyclic or sawtooth K/V scans) and of its L2 sector model, written from the
paper and independent of the CUDA path: no shared kernels, headers, helpers or tables.
"""
