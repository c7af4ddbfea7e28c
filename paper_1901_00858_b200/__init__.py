"""B200-native FP16 convolution layer forward (Caffe semantics) behind a small C ABI.

`workloads` (seeded synthetic inputs) imports without the CUDA library; everything in
`binding` needs the compiled library and fails loudly if it is missing.
"""
__all__ = ["workloads", "binding"]
