"""B200-native group-wise mixed-precision weight-only linear layer (SliM-LLM hot path).

The compute lives in a C-ABI CUDA library (csrc/, declared in include/slim.h);
`binding` marshals arguments to it.  `workloads` draws seeded synthetic inputs.
Importing this package does not load the CUDA library; the first call does, and
fails loudly if the library has not been built.
"""
