"""B200-native batched fixed-point Pong environment step (CUDA, sm_100a).

`paper_2603_12145_b200.pong` is the binding of the C-ABI library declared in
include/pong.h; `paper_2603_12145_b200.build` compiles it; `inputs` holds the
seeded synthetic input generators.  Importing the package loads nothing.
"""
__all__ = ["pong", "cartpole", "build", "inputs", "sharding", "verify"]
