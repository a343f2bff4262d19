"""Forward convolutional layers of a CNN (SqueezeNet v1.0) as sm_100a CUDA kernels
behind a C-ABI library.  `binding` is the thin ctypes face of that library;
`synth` draws the seeded synthetic inputs used by tests and benchmarks."""
