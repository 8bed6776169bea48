"""CPU oracle for PEVLM prefill attention (fp64).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's cpu_baseline / reference legs may import
this package; the product path (the CUDA library and its binding) never does.  It imports
nothing from the CUDA package.

`oracle.api`   ctypes wrapper over the C oracle (pevlm_oracle.c)
`oracle.dense` a second, independent numpy evaluation through a materialised dense mask
"""
