"""B200-native Switch FFN layer (Switch Transformer, arxiv 2101.03961): ctypes binding over libswitch_moe.so.

`paper_2101_03961_b200.switch_moe` holds the entry points; `paper_2101_03961_b200.inputs` the seeded synthetic
input generators; `paper_2101_03961_b200.build` compiles the CUDA library in-tree.
"""
