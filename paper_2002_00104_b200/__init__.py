"""B200-native PWLQ hot path: abs-max, breakpoint search, quantize, dequantize."""
