"""B200-native paged decode attention (split-KV, GQA) behind a C ABI.

`paper_2609_37062_b200.binding` loads the CUDA library and mirrors its entry
points; `paper_2609_37062_b200.workloads` builds seeded synthetic inputs.
There is no CPU implementation in this package: importing `binding` without
the built library raises.
"""

__all__ = ["binding", "workloads", "build"]
