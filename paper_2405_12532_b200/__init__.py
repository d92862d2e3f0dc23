"""PyramidInfer's prefill selection hot path for B200 (sm_100a).

The CUDA library `libpyr.so` (built in-tree from csrc/) holds every step of the
path; `binding` marshals arguments to its C ABI. There is no CPU fallback: a
call without the built library raises.
"""
