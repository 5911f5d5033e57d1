"""B200-native layout-driven Muon step (momentum, Newton-Schulz, update, flat-shard gather/scatter).

`workloads` describes synthetic inputs; `binding` marshals arguments into the C-ABI
library built from `csrc/`.  Nothing here computes: every step runs in the CUDA kernels.
"""
__all__ = ["workloads", "binding", "build"]
