"""B200-native layout-driven Muon step (momentum, Newton-Schulz, update, flat-shard gather/scatter).

`workloads` describes synthetic inputs; `binding` marshals arguments into the C-ABI
library built from `csrc/`; `optim.Muon` is a torch.optim front end on top of the binding.  Nothing here computes: every step runs in the CUDA kernels.
"""
__all__ = ["workloads", "binding", "build", "optim"]
