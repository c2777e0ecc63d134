"""TEST INFRASTRUCTURE ONLY -- CPU oracles written from the paper.

``oracle.cnn``    : Eq. 1 (the seven-nested-loop CNN) in fp64, plain C behind ctypes.
``oracle.bounds`` : Theorem 1 terms, the Section-5 tiling LP, Theorem 2's case tree.
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
"""
