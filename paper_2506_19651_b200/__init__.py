"""B200-native (sm_100a) PEVLM prefill attention: hand-written CUDA kernels behind a C-ABI
library, with a thin ctypes binding (`paper_2506_19651_b200.binding`).

Importing the package does not load the CUDA library; `binding.lib()` does, and fails
loudly if the library has not been built (`python -m paper_2506_19651_b200.build`).
"""
