"""MVUE N:M gradient pruning and 2:4-sparse GEMMs for NVIDIA B200 (sm_100a).

The compute lives in the CUDA library under `csrc/`; `binding` loads it through
its C ABI.  There is no CPU fallback: any call raises if the library is absent.
"""
