"""B200-native kernels for the token-level policy-loss pass of Mutual RL (GRPO / PRP / XGRPO / SGT).

The product is the C-ABI library `libmrl.so` (declared in `include/mrl.h`); `binding` is a thin
ctypes layer over it with the same names, and `synth` draws the seeded synthetic inputs.
"""
