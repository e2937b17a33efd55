"""B200-native (sm_100a) ZigzagAttention inference hot path.

`binding` is the ctypes front end of the C-ABI CUDA library (`libzigzag_b200.so`, built
by `build.build()`); `inputs` draws the seeded synthetic workloads.  Nothing here falls
back to a CPU implementation: using `binding` without the built library raises.
"""
__all__ = ["binding", "build", "inputs"]
