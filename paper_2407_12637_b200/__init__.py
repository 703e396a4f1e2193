"""B200-native quantized backward pass of arXiv 2407.12637 (INT4 fixed-point training).

`lbt`     -- thin ctypes binding of the C-ABI CUDA library (argument marshalling only).
`synth`   -- seeded synthetic inputs shaped like the paper's CNN workloads.
`shapes`  -- the layer shapes of the benchmark configurations.
`build`   -- compiles the CUDA library for sm_100a.

Nothing here imports a CPU implementation of the method; the CUDA library is
loaded on first use of `lbt` and its absence is an error.
"""
__all__ = ["lbt", "synth", "shapes", "build"]
