"""Mixed-precision cached embedding training step for B200 (sm_100a).

The hot path lives in the CUDA library built from csrc/ and is reached through
the C ABI declared in include/mpe.h; `binding` marshals arguments to it.
"""
