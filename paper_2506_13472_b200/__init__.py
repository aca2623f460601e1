"""B200-native ROSAQ hot path: calibration Gram matrix, rotate + mixed-precision quantize,
and the fused rotated mixed-precision linear, as hand-written sm_100a CUDA behind a C ABI
(include/rosaq.h).  `binding` is the ctypes front end; `synth` holds the seeded synthetic
inputs; `pca` is the host eigensolve between the calibration and quantization calls."""

__all__ = ["binding", "synth", "pca", "build"]
