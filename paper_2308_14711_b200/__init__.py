"""Hard-routed inference for Fast Feedforward networks on B200 (sm_100a).

`workloads` draws the synthetic inputs; `binding` is the thin ctypes layer over
the C-ABI CUDA library (libfff.so).  Nothing is loaded at import time; the
binding raises if the CUDA library has not been built.
"""
