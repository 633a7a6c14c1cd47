"""B200-native hot path of SNIP's mixed-precision linear layer (quantizers, block-scaled GEMMs,
error-norm statistics).  `api` is the thin binding over the C-ABI library; `workloads` draws the
seeded synthetic inputs.  There is no CPU fallback: importing `api` without the built CUDA
library raises."""

__all__ = ["api", "workloads", "build"]
