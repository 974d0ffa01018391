"""B200-native MRP drafting step: C-ABI CUDA library plus a thin Python binding."""
__version__ = "0.1.0"
