"""B200-native per-chunk KV-cache step of StreamingVLM-style streaming inference.

`streamgen` (synthetic inputs) imports nothing else; the CUDA binding lives in `binding` and is
loaded lazily so that the input generator can be used on machines without the built library.
"""

# Path of an alternative build of the C-ABI library for `binding` to load instead of libsvlm.so, set by a
# program BEFORE it imports `binding` (the benchmark's decode-trace workload points it at the instrumented
# build).  None: the product library.
LIB_OVERRIDE = None
