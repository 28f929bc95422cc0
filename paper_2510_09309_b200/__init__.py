"""MaskKV compress-and-attend path for NVIDIA B200: hand-written sm_100a kernels behind a C ABI
(include/maskkv.h), a ctypes binding (`binding`), seeded synthetic inputs (`synth`) and the in-tree
build (`build`).  Importing the package is cheap; `binding` loads the shared library and fails loudly
when it has not been built."""
__all__ = ["binding", "build", "synth"]
