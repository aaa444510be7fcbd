"""CPU oracle for the coded-gradient hot path.

TEST INFRASTRUCTURE ONLY. Plain, slow, obviously-correct restatements of what
the paper defines, used by the tests, by the smoke check and by the benchmark's
CPU-baseline leg. The product package never imports this package, and this
package never imports the product.

  roundpath.py / agc_oracle.c  per-round path in IEEE binary32 (encode, bucket
                               norm, stochastic rounding, packing, decode,
                               update), C compiled with gcc by build.py
  design.py                    design-time quantities in float64 (Theorem 1
                               structure, interval construction, support-
                               restricted code, unbiasedness check, error
                               bounds, DP and low-complexity bit allocation,
                               two-track decoder)

Pins: every function here is checked in tests/ (-m "not gpu") against facts
the paper or the mathematics fix. The one exception is stated where it occurs:
exact agreement of `design.bit_allocate_low_complexity` with the authors' own
allocator is "parity unpinned" (the paper under-specifies two of its steps);
its outputs are pinned only through properties and against the exact DP.
"""
