"""B200-native inverse of a masked k x k convolution with parallel backpropagation.

The hot path lives in the CUDA library built from `csrc/` (C ABI declared in
`include/invconv.h`); `binding` is its thin ctypes front end and `workloads`
draws the seeded synthetic inputs.  Importing the package itself loads neither
torch nor the shared library.
"""
__version__ = "0.1.0"
