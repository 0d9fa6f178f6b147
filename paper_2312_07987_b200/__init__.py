"""B200-native forward pass of one SwitchHead attention layer.

`inputs` (seeded synthetic workloads) imports without the CUDA library; `binding`
(the ctypes layer over libswitchhead.so) loads it and fails loudly if it is missing.
"""
