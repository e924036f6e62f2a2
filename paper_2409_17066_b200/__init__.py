"""B200-native (sm_100a) inference hot path of VPTQ: the fused vector-quantized linear layer.

`binding` wraps the C ABI of libvptq.so (include/vptq.h); `synth` draws the seeded
synthetic workloads; `build` compiles the library in-tree.
"""
