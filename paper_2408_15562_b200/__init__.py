"""B200-native tree-verification step of lossless speculative decoding.

Three operations, each a hand-written sm_100a kernel behind a C-ABI library
(`include/fspad.h`): tree-masked verify attention, lossless tree acceptance
(greedy or recursive rejection sampling) and accepted-path KV compaction.

`paper_2408_15562_b200.binding` is the thin ctypes layer over that library;
`paper_2408_15562_b200.synth` generates the seeded synthetic workloads.
Importing this package loads nothing native: the library is opened on first
use of the binding and a missing build raises immediately.
"""

__all__ = ["binding", "synth", "build"]
