"""B200-native (sm_100a) quantize / dequantize for the Adaptive Block-Scaled (IF) data types.

The CUDA library is loaded on first use of :mod:`paper_2603_28765_b200.binding`; importing the
package itself (for example for :mod:`paper_2603_28765_b200.inputs`) loads nothing native.
"""
__all__ = ["inputs", "binding", "build"]
