"""B200-native AMS KV-compression step: Python face of the C-ABI library.

`inputs` builds seeded synthetic workloads; `binding` marshals arguments into
`libams.so` (every step of the path runs in the library's CUDA kernels).  The
library is loaded on first use and its absence is an error: there is no CPU
fallback.
"""
__all__ = ["inputs", "binding", "build"]
