"""B200-native A2SGD per-worker gradient path (two-level gradient averaging).

``binding`` wraps the C-ABI CUDA library (``liba2sgd.so``, built in-tree from
``csrc/``); ``workloads`` holds the seeded synthetic input generators.  There
is no CPU fallback: calling the binding without the built library raises.
"""
