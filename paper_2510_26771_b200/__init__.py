"""B200-native STaMP-quantized linear layer (sequence transform + mixed-precision
activation quantization + int8 tensor-core GEMM + inverse transform).

The CUDA library is loaded lazily by `paper_2510_26771_b200.binding`; importing this
package (e.g. for the seeded input generators) does not need a GPU.
"""
