"""B200-native STTM token merging: a C-ABI CUDA library (libsttm.so) and its binding.

``inputs`` (seeded synthetic videos) imports nothing from the CUDA side.  ``binding``
loads the library lazily and raises when it is missing: there is no CPU fallback.
"""
__all__ = ["inputs", "binding", "build", "shard"]
