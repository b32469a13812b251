"""B200-native paged-KV offload path (the data path EfficientAgent's host tier drives).

``eakv`` is the ctypes binding of the C-ABI library ``libeakv.so`` (hand-written CUDA for
sm_100a plus a C++ control plane); ``harness`` drives whole agent turns through it with
PyTorch used only for device memory and streams.  Importing this package loads nothing;
``eakv.lib()`` loads the shared library and fails loudly when it has not been built.
"""
__all__ = ["eakv", "build", "harness", "replay", "capacity", "multi"]
