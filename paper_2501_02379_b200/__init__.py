"""B200-native TensorGRaD optimizer step (sparse + low-rank Tucker gradient
compression with Adam in the compressed space) behind a C ABI.

`synth` generates seeded inputs (numpy only); `binding` loads the CUDA
library lazily and raises if it is missing -- there is no CPU fallback.
"""
