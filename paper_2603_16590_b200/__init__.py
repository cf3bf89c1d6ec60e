"""B200-native W4A4 linear hot path of BATQuant: CUDA kernels behind a C-ABI
(``include/batq.h``), a ctypes binding with the same names (``binding``) and
seeded synthetic inputs (``synth``)."""
