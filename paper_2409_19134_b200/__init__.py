"""B200-native partitioned decode attention (Secure Partitioned Decoding hot path).

`workloads` builds seeded synthetic inputs; `binding` is the thin ctypes layer over the
C-ABI library `libspd.so` built from `csrc/`.  Importing this package loads nothing
native; the first call into `binding` loads the library and fails loudly if it is absent.
"""
__all__ = ["workloads", "binding"]
