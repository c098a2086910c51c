"""B200-native FFD sparse decode attention: C-ABI CUDA library + thin binding (see ``ffd.py``)."""
