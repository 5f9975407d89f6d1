"""DiffQKV attention over the KV cache, hand-written CUDA for sm_100a behind a C ABI.

``paper_2501_13629_b200.api`` is the ctypes binding of ``libdiffqkv.so`` (it raises at
import when the library has not been built); ``paper_2501_13629_b200.workloads`` makes the
seeded synthetic inputs.  Importing the package itself loads nothing.
"""
__version__ = "0.1.0"
