"""ExCP checkpoint compression hot path for B200 (sm_100a): CUDA kernels behind a
C ABI, with a thin Python binding.  `synth` makes seeded test inputs."""
