"""APAR decode hot path for NVIDIA B200: fork, KV append and tree decode attention over a
paged KV cache with shared ancestor blocks.  The work is done by libapar.so (CUDA, sm_100a);
this package only marshals arguments.  `synth` holds the seeded synthetic workloads."""
