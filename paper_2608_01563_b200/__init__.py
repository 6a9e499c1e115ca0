"""B200-native scaled-dot-product attention forward + backward (C-ABI CUDA library
``libmgn_attn.so`` plus a thin ctypes binding).  See ``binding.py``."""
