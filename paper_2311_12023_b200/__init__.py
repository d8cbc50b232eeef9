"""B200-native LQ-LoRA linear layer: packed NormalFloat weights + low-rank term.

``inputs`` holds the seeded synthetic generators (numpy only); ``binding`` is the thin
ctypes layer over ``liblqlora.so`` (imported lazily because it needs torch and the
compiled library).
"""

__all__ = ["inputs", "binding", "build"]
