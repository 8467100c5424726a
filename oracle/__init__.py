"""CPU oracle for RIB window attention.  TEST INFRASTRUCTURE ONLY.

A plain fp64 restatement of the paper's definition (Eq. 5, Eq. 6, SoftMax(S)V and its chain
rule).  It may be imported by the tests, by the smoke check and by the CPU-baseline leg of the
benchmark, and by nothing else; the CUDA library never calls it and shares no code with it.
"""
