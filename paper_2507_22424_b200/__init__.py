"""B200 (sm_100a) tree-verification path of Spec-VLA behind a C ABI (include/specvla.h).

`binding` loads libspecvla.so and marshals arguments; every step of the path runs in the
library's CUDA kernels. There is no CPU fallback: importing `binding` raises if the library
has not been built (see build.py).
"""
