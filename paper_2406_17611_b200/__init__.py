"""VARCO partitioned graph-convolution layer with variable-rate halo compression,
hand-written CUDA for sm_100a behind a C-ABI library.

``synth`` holds the seeded input generators; ``binding`` loads the compiled
library (``libvarco.so``) and mirrors its entry points.  Nothing here falls
back to the CPU: without the compiled library the binding raises.
"""
