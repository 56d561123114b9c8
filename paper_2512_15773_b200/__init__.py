"""B200-native TS-DP speculative denoising loop (arXiv 2512.15773): CUDA library + thin binding.

`binding` wraps libtsdp.so (C ABI in include/tsdp.h); `inputs` holds the seeded synthetic inputs;
`build` compiles the library in-tree for sm_100a."""
