"""B200-native exact-attention response replay (LongStraw hot path).

`workloads` draws the seeded synthetic inputs; `binding` is the thin ctypes
layer over the C-ABI library built from `csrc/` (see `build.build_library`).
"""
