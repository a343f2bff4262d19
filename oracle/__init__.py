"""CPU oracle (test infrastructure only).

A plain, slow, obviously-correct implementation of the forward layers the
CUDA library computes, written from the paper's definitions.  Only tests,
the smoke check and the benchmark's CPU-baseline leg may import this package;
the CUDA path never does, and this package never imports the CUDA path.
"""
