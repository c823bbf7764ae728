"""B200-native MeteoRA linear forward: y = W0 x + sum_{i in topk(x)} w_i(x) B_i (A_i x).

The compute lives in the CUDA library built from `csrc/` (C ABI declared in
`include/meteora.h`); `binding` marshals torch tensors into it and `workloads`
draws the seeded synthetic inputs.  Importing the package does not load the
library; the first call does, and raises if it has not been built.
"""
__all__ = ["binding", "workloads"]
