"""B200-native paged decode attention + KV append behind the `ooco_*` C ABI.

`inputs` holds the seeded synthetic batches, `binding` the ctypes access to the CUDA
library (imported lazily: it needs the built shared object), `build` the nvcc step.
"""
__all__ = ["inputs", "binding", "build"]
