"""B200-native Plan-Verify-Fill (PVF) vocabulary pass: a C-ABI CUDA library (``csrc/``), its thin
ctypes binding (``binding``) and the seeded synthetic-input generator (``synth``).

Importing the package loads nothing; ``binding`` loads the CUDA library on first use and raises
if it has not been built."""
