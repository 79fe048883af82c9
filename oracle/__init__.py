"""CPU oracle for streamlined few-bit QNN inference -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It shares no code with the CUDA path and never imports it.

Contents
--------
qnn_oracle.c   plain C loops: integer GEMM, thresholding, direct convolution,
               max-pool (compiled by ``oracle.build``).
oracle.py      ctypes access to the C functions on numpy arrays.
bitserial.py   the bit-plane identity of Section 3.1 (Algorithms 1-2) on Python integers,
               one big integer per plane row (tiny sizes only; pins the GEMM oracle).
planeskip.py   bit-plane products without the low-order plane pairs (the paper's
               conclusion: approximate computing from the higher-order bits), numpy int64.
streamline.py  float batch-norm + quantizer reference and the threshold
               absorption of Section 2.1 (fp64).
alexnet.py     the AlexNet-shaped layer chain of Section 4.2 built from the above.
"""
