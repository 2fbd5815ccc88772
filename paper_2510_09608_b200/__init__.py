"""B200-native per-chunk KV-cache step of StreamingVLM-style streaming inference.

`streamgen` (synthetic inputs) imports nothing else; the CUDA binding lives in `binding` and is
loaded lazily so that the input generator can be used on machines without the built library.
"""
