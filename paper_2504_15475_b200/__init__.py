"""libersd: exponential-race speculative decoding on one B200 (sm_100a).

``workloads`` makes the seeded synthetic inputs.  ``binding`` loads the CUDA
library ``libersd.so`` and exposes its C entry points under the same names;
it raises at load time when the library has not been built -- there is no CPU
fallback.
"""
__all__ = ["workloads", "binding"]
