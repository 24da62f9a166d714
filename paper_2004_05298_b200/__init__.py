"""B200-native (sm_100a) DEF / DEF-A / EF optimizer step with random block-wise
gradient sparsification.  The work is done by the C-ABI library built from csrc/
(declared in include/def.h); `binding` marshals torch tensors into it and `workloads`
draws the synthetic inputs.  Importing the package loads nothing heavy; the CUDA
library is opened on first use and its absence is an error, never a fallback."""

__all__ = ["binding", "workloads", "build"]
