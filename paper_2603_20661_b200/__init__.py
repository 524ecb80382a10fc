"""B200-native batched simulation of the WWW.Serve decentralized serving network.

`paper_2603_20661_b200.synth` builds seeded inputs and loads no native code;
`paper_2603_20661_b200.binding` is the thin ctypes layer over the C-ABI CUDA
library (`libwwws.so`, built in-tree by `paper_2603_20661_b200.build`).  There is
no CPU implementation in this package: without the CUDA library the binding
raises.
"""
