"""B200-native Orth-Dion / Dion optimizer step (C-ABI library + thin Python binding).

`workloads` (synthetic inputs) is importable without the CUDA library; everything in
`binding` loads `liborthdion.so` on first use and raises if it is missing.
"""
