"""B200-native LASER-KV prefill-time token selection: ctypes binding over a C-ABI CUDA library."""
__version__ = "0.1.0"
