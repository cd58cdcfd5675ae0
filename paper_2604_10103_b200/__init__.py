"""B200-native hybrid attention (block-sparse sliding-window attention + linear history state).

The compute lives in ``libhf.so`` (CUDA, sm_100a, C ABI declared in ``include/hf.h``);
``binding`` marshals arguments into it and ``inputs`` generates seeded synthetic tensors.
Importing the package does not load the library; ``binding.lib()`` does, and raises if it
is missing -- there is no CPU fallback.
"""
__all__ = ["inputs", "binding", "build"]
