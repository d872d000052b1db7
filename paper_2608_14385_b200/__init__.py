"""B200-native decode forward of one DeaMoE layer (two-stage department/expert routing).

`paper_2608_14385_b200.binding` is the thin ctypes layer over the C-ABI library
(`libdeamoe.so`, hand-written sm_100a CUDA); `paper_2608_14385_b200.synth` makes
seeded synthetic layers.  There is no CPU fallback: using the binding without the
built library raises.
"""
