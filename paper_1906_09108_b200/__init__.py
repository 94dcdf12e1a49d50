"""B200-native FDG (fully decoupled training with delayed gradients) module-step:
libfdg.so (hand-written CUDA for sm_100a behind a C ABI, see include/fdg.h) and its
thin ctypes binding.  `from paper_1906_09108_b200 import binding`."""
