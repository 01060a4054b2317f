"""B200-native selective Jacobi decoding for TarFlow-style autoregressive flows.

`synth` (seeded inputs) imports without the CUDA library; `binding` loads
``libtarflow.so`` and fails loudly when it is missing.
"""
