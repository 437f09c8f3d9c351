"""B200-native draft-verification step of Hierarchical Speculative Decoding.

`inputs` (seeded synthetic workloads), `roofline` (algorithmic work per step) and `shard`
(region sharding across replicas) are pure host code.  `binding` loads the CUDA C-ABI
library and raises if it is missing: there is no CPU fallback.
"""
__all__ = ["inputs", "roofline", "shard", "binding", "runtime"]
