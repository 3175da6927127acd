"""B200-native SP-KV (Self-Pruned Key-Value attention) decode path.

``spkv`` is the thin ctypes binding over the C-ABI CUDA library (``libspkv.so``);
``synth`` holds the seeded synthetic-workload generators.
"""
