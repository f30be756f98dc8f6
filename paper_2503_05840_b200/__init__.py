"""B200-native K-cache-only ("slim") multi-head decode attention.

`binding` mirrors the C ABI of libslim.so (include/slim.h); `layer.SlimLayer`
owns the torch buffers for one layer; `synth` draws seeded synthetic inputs;
`build` compiles the library in-tree.  Nothing here computes attention on the
CPU: without the CUDA library and a CUDA device the calls raise."""
__all__ = ["binding", "layer", "synth", "build"]
