"""B200-native (sm_100a) hot path of an OrbitQuant quantized linear layer.

`binding` wraps the C-ABI library liboq.so (built by `build`); `synth` holds the seeded input
generators.  Importing the package loads nothing; the library is loaded on first use.
"""
