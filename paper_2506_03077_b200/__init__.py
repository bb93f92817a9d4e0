"""B200-native streamed backward (StreamBP) for decoder-only transformers.

`synth` builds seeded synthetic inputs; `binding` loads the C-ABI CUDA library
(`libstreambp.so`, built by `build.py`) and exposes its entry points under the
same names.  Importing the package does not load the CUDA library.
"""
__all__ = ["synth"]
