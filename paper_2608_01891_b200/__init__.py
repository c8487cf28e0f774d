"""B200-native A/F decode-layer hot path (attention side + FFN side + interleave).

`inputs` holds the seeded synthetic workload generators; `aflex` is the thin
ctypes binding over the C-ABI CUDA library (`include/aflex.h`)."""
