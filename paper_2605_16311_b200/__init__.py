"""SignMuon optimizer step for NVIDIA B200 (sm_100a): hand-written CUDA kernels behind a C ABI.

`paper_2605_16311_b200.binding` is the thin ctypes layer over the shared library
(argument marshalling only); `paper_2605_16311_b200.workloads` holds the seeded
synthetic inputs.  Importing the package does not load the native library; the
first use of the binding does, and raises if it has not been built.
"""
__all__ = ["binding", "workloads", "build"]
