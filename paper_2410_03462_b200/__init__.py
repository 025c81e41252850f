"""GRF-masked linear attention on B200: a C-ABI CUDA library (csrc/, include/grf.h) and its ctypes binding.

`binding` mirrors the C entry points one to one; `api` adds a small object layer that owns the
device buffers (torch tensors) around them.  There is no CPU fallback: importing `binding` loads
libgrf.so or fails."""
