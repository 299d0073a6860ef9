"""B200-native sparse decode hot path (score -> per-KV-head top-k -> host gather -> GQA decode attention).

`workloads` draws seeded inputs; `binding` is the thin ctypes layer over the
C-ABI library built from `csrc/` (it raises if the library is missing: there is
no CPU fallback).
"""
