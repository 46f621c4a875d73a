"""B200-native DynamicKV prefill-time KV-cache compression (arXiv 2412.14838).

``synth``   seeded synthetic inputs (pure data, no method arithmetic)
``binding`` ctypes view of the C-ABI library ``libdkv.so`` (built by ``build.py``)

Importing the package loads nothing native; ``binding.load()`` does, and fails loudly when the
CUDA library has not been built.
"""
