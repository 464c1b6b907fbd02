"""Task-KV (arXiv 2501.15113) hot path for NVIDIA B200: a C-ABI CUDA library
(`libtaskkv.so`, declared in include/taskkv.h) and its ctypes binding.

`workloads` (seeded synthetic inputs) imports without the library; `binding`
and `configs` need the built library and raise if it is missing."""
