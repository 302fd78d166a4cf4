"""B200-native ARMOR block coordinate descent: CUDA kernels behind a C ABI, plus a ctypes binding.

Importing the package loads nothing native; `paper_2510_05528_b200.binding` opens the shared
library on first use and raises if it has not been built."""
