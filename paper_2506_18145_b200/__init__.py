"""B200 (sm_100a) forward pass of one Routing-Mamba (RoM) layer: hand-written CUDA kernels behind a
small C ABI (include/rom.h), with a ctypes binding (`binding`) and seeded synthetic inputs (`synth`).
Importing the package does not load the CUDA library; `binding.lib()` does, and fails if it is absent."""
