"""libtlin: exact-softmax attention of TLinFormer's connectivity on B200 (sm_100a).

``synth`` makes seeded inputs; ``binding`` is the ctypes layer over the C-ABI in
``include/tlin.h``.  Nothing here computes attention on the CPU: if the CUDA
library is missing the binding raises.
"""
