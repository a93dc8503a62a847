"""CPU oracle (test infrastructure only).

Plain, slow restatement of what the CUDA library must compute.  Only the test
suite, the smoke check and the CPU-baseline leg of the benchmark may import
this package; the product never does.
"""
