"""B200-native per-user segment encryption with ownership labels (GIFT hot path).

`workloads` holds the seeded input generators; `binding` is the thin ctypes layer over
the C-ABI library built from `csrc/`.  Importing the package does not load the library;
the first binding call does, and fails loudly if it has not been built.
"""
