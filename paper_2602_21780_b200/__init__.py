"""B200-native compressed-KV streaming attention step (XStreamVGGT hot path).

The product is the C-ABI library built from csrc/ (see include/xsv.h); this
package holds its thin ctypes binding (`binding`) and the seeded synthetic
input generators (`synth`).  Nothing is loaded at import time: the binding
loads the shared library on first use and fails loudly if it is missing.
"""
