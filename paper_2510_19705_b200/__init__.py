"""B200-native hot path of Hierarchical Speculative Decoding (HSD).

``paper_2510_19705_b200.binding`` is the thin ctypes layer over the C-ABI library
(``include/hsd.h``); ``paper_2510_19705_b200.inputs`` holds the seeded synthetic input
generators and the benchmark shapes; ``paper_2510_19705_b200.build`` compiles the
library in-tree.  Nothing is imported eagerly: loading the shared library happens on
first use of the binding and fails loudly when it has not been built.
"""
