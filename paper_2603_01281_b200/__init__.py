"""B200-native SEKA / AdaSEKA steered prefill attention (C-ABI CUDA library + thin binding).

``inputs`` (seeded synthetic workloads) imports nothing else from this package;
the binding in ``binding`` loads the compiled CUDA library lazily and raises if
it is missing -- there is no CPU fallback.
"""
