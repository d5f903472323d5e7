"""B200-native PatchKV patch construction.

Sub-modules
-----------
inputs   seeded synthetic workloads (the five benchmark configs); numpy only, none of the
         method's arithmetic, shared by the tests' CPU checker and the CUDA path.
binding  thin ctypes marshalling over the C-ABI library ``libpkv.so`` (pkv_build_patch,
         pkv_merge, ...).  Every step of the path runs in the library's CUDA kernels; the
         binding raises if the library is missing.
build    nvcc driver that compiles ``csrc/*.cu`` for sm_100a into ``libpkv.so`` in-tree.

Nothing is imported eagerly so that ``inputs`` can be used without the CUDA library.
"""

__all__ = ["inputs", "binding", "build"]
