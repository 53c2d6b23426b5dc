"""B200-native fused attention with a Jacobian-vector product and its backward pass.

The compute lives in a C-ABI CUDA library (csrc/, built for sm_100a); `binding` marshals
arguments to it.  Nothing here falls back to a CPU or library implementation: calling an op
without the built library raises.
"""
