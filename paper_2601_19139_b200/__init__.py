"""B200 decode-step library for 4-bit group-quantised models over a paged KV pool.

`binding` forwards to the C ABI of libq4decode.so (include/q4decode.h); `build`
compiles it.  Nothing is loaded at import time.
"""
__all__ = ["binding", "build"]
